// Window importance scoring and ratio-driven selection (MixA-Q Section 3.2; pruned class: Section 3.4).
// Integer work throughout: int8 score codes, int32 token energies, int64 window scores, ranks by counting.
#include "kernels.h"

namespace mixaq {

// energy[token] = sum_c clamp(rne(x*inv), -127, 127)^2.  Integer sums are exact in any order, so the loads are
// laid out for the memory system only: a group of G = 8 lanes owns one token and walks its channels with
// 16-byte loads (C is a multiple of 32), four tokens per warp.
__device__ __forceinline__ int score_code_sq(float v, float inv) {
  // clamp before rounding (the bounds are integers), then round to nearest-even by the 1.5*2^23 addition
  float t = fminf(fmaxf(__fmul_rn(v, inv), -127.0f), 127.0f);
  int code = (int)(__float_as_uint(__fadd_rn(t, 12582912.0f)) - kMagicBits);
  return code * code;
}
__global__ void __launch_bounds__(256) k_energy(const float* __restrict__ x, int32_t* __restrict__ energy,
                                                long ntok, int C, float inv) {
  const long tok = ((long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;
  const int sub = threadIdx.x & 7;
  int e = 0;
  if (tok < ntok) {
    const float4* row = reinterpret_cast<const float4*>(x + tok * C);
    for (int c0 = sub; c0 < C / 4; c0 += 32) {          // four loads in flight per lane
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = c0 + 8 * u < C / 4 ? __ldg(row + c0 + 8 * u) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        e += score_code_sq(v[u].x, inv) + score_code_sq(v[u].y, inv) + score_code_sq(v[u].z, inv) + score_code_sq(v[u].w, inv);
    }
  }
#pragma unroll
  for (int off = 4; off >= 1; off >>= 1) e += __shfl_xor_sync(0xffffffffu, e, off);
  if (sub == 0 && tok < ntok) energy[tok] = e;
}

__device__ __forceinline__ int window_src(int b, int H, int W, int Hp, int Wp, int shift, int nwx, int w, int t) {
  int wy = w / nwx, wx = w - wy * nwx;
  int i = t / WS, j = t - i * WS;
  int y = wy * WS + i + shift; if (y >= Hp) y -= Hp;
  int x = wx * WS + j + shift; if (x >= Wp) x -= Wp;
  if (y >= H || x >= W) return -1;
  return (b * H + y) * W + x;
}

// One warp per (image, window): score = sum of the energies of the window's real tokens under this
// block's own (possibly shifted, cyclically wrapped) partition.
constexpr int MAX_SELECT_BATCH = 24;
struct SelectBatch { SelectArgs a[MAX_SELECT_BATCH]; };

__global__ void __launch_bounds__(256) k_window_score(const __grid_constant__ SelectBatch batch) {
  const SelectArgs& a = batch.a[blockIdx.y];
  int gw = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int lane = threadIdx.x & 31;
  if (gw >= a.B * a.nW) return;
  int b = gw / a.nW, w = gw - b * a.nW;
  int Hp = (a.H + WS - 1) / WS * WS, Wp = (a.W + WS - 1) / WS * WS;
  long long s = 0;
  for (int t = lane; t < WT; t += 32) {
    int src = window_src(b, a.H, a.W, Hp, Wp, a.shift, a.nwx, w, t);
    if (src >= 0) s += a.energy[src];
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
  if (lane == 0) a.score[gw] = s;
}

// Rank by counting: rank(w) = #{v : v precedes w in (score desc, index asc)}; ranks are a permutation.
// One warp per window: the lanes split the windows to compare against, the counts are summed over the warp,
// and the lanes then write the batch bookkeeping of the window's slot (49 source-token indices) together.
constexpr int RANK_WARPS = 8;
__global__ void __launch_bounds__(RANK_WARPS * 32) k_rank_emit(const __grid_constant__ SelectBatch batch) {
  extern __shared__ long long s_score[];
  const SelectArgs& a = batch.a[blockIdx.z];
  const int b = blockIdx.y;
  const int64_t* sc = a.score + (long)b * a.nW;
  for (int i = threadIdx.x; i < a.nW; i += blockDim.x) s_score[i] = sc[i];
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int w = blockIdx.x * RANK_WARPS + (threadIdx.x >> 5);
  if (w >= a.nW) return;
  const long long mine = s_score[w];
  int cnt = 0;
  if (!a.reverse) {
    for (int v = lane; v < a.nW; v += 32) { long long o = s_score[v]; cnt += (o > mine) || (o == mine && v < w); }
  } else {
    for (int v = lane; v < a.nW; v += 32) { long long o = s_score[v]; cnt += (o < mine) || (o == mine && v < w); }
  }
  const int rank = __reduce_add_sync(0xffffffffu, cnt);
  const int c = rank < a.n_hi ? 0 : (rank < a.n_hi + a.n_lo ? 1 : 2);
  const int Hp = (a.H + WS - 1) / WS * WS, Wp = (a.W + WS - 1) / WS * WS;
  int32_t* dst; long slot;
  if (c == 0)      { slot = (long)b * a.n_hi + rank;                     dst = a.rowsrc_hi; }
  else if (c == 1) { slot = (long)b * a.n_lo + (rank - a.n_hi);          dst = a.rowsrc_lo; }
  else             { slot = (long)b * a.n_pr + (rank - a.n_hi - a.n_lo); dst = a.rowsrc_pr; }
  if (lane == 0) {
    a.order[(long)b * a.nW + rank] = w;
    a.cls[(long)b * a.nW + w] = (uint8_t)c;
    if (c == 0) a.win_hi[slot] = w;
    else if (c == 1) a.win_lo[slot] = w;
  }
  for (int t = lane; t < WT; t += 32) dst[slot * WT + t] = window_src(b, a.H, a.W, Hp, Wp, a.shift, a.nwx, w, t);
}

// One warp per (image, class): walks the windows in ascending index, 32 at a time, and appends the members of its class
// (order-preserving compaction by ballot).
struct ClassListArgs { const uint8_t* cls; int32_t* out[3]; int count[3]; int B, nW; };
__global__ void __launch_bounds__(96) k_class_lists(ClassListArgs a) {
  const int b = blockIdx.x, c = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int32_t* out = a.out[c];
  if (!out) return;
  out += (long)b * a.count[c];
  const uint8_t* cls = a.cls + (long)b * a.nW;
  int base = 0;
  for (int w0 = 0; w0 < a.nW; w0 += 32) {
    const int w = w0 + lane;
    const bool mine = w < a.nW && cls[w] == c;
    const unsigned m = __ballot_sync(0xffffffffu, mine);
    if (mine) out[base + __popc(m & ((1u << lane) - 1u))] = w;
    base += __popc(m);
  }
}

void launch_class_lists(const uint8_t* cls, int B, int nW, int32_t* const out[3], const int count[3], cudaStream_t st) {
  ClassListArgs a;
  a.cls = cls; a.B = B; a.nW = nW;
  for (int c = 0; c < 3; ++c) { a.out[c] = out[c]; a.count[c] = count[c]; }
  k_class_lists<<<B, 96, 0, st>>>(a);
  ++g_launches;
}

void launch_energy(const float* x, int32_t* energy, long ntok, int C, float inv_scale, cudaStream_t st) {
  k_energy<<<(unsigned)((ntok * 8 + 255) / 256), 256, 0, st>>>(x, energy, ntok, C, inv_scale);
  ++g_launches;
}

void launch_select(const SelectArgs* args, int count, cudaStream_t st) {
  // all entries share B, H, W (one stage); shift, ratios and output buffers differ
  for (int first = 0; first < count; first += MAX_SELECT_BATCH) {
    const int n = count - first < MAX_SELECT_BATCH ? count - first : MAX_SELECT_BATCH;
    SelectBatch batch;
    for (int i = 0; i < n; ++i) batch.a[i] = args[first + i];
    for (int i = n; i < MAX_SELECT_BATCH; ++i) batch.a[i] = args[first];
    const SelectArgs& a = args[first];
    const int nwin = a.B * a.nW;
    k_window_score<<<dim3((nwin + 7) / 8, n), 256, 0, st>>>(batch);
    ++g_launches;
    dim3 grid((a.nW + RANK_WARPS - 1) / RANK_WARPS, a.B, n);
    k_rank_emit<<<grid, RANK_WARPS * 32, (size_t)a.nW * sizeof(long long), st>>>(batch);
    ++g_launches;
  }
}

// ---- guard zones ---------------------------------------------------------------------------------------
namespace {
constexpr int GUARD_BATCH = 48;
constexpr uint32_t GUARD_PATTERN = 0xA5C3E1B7u;
struct GuardList { uint32_t* zone[GUARD_BATCH]; };
template <bool FILL>
__global__ void k_guards(GuardList g, int* status) {
  uint32_t* z = g.zone[blockIdx.x];
  const int i = threadIdx.x;                               // GUARD_BYTES / 4 threads
  if (FILL) z[i] = GUARD_PATTERN ^ (uint32_t)i;
  else if (z[i] != (GUARD_PATTERN ^ (uint32_t)i)) atomicOr(status, 2);
}
}  // namespace

void launch_guards(void* const* zones, int count, bool fill, int* status, cudaStream_t st) {
  for (int first = 0; first < count; first += GUARD_BATCH) {
    const int n = count - first < GUARD_BATCH ? count - first : GUARD_BATCH;
    GuardList g;
    for (int i = 0; i < GUARD_BATCH; ++i) g.zone[i] = (uint32_t*)zones[first + (i < n ? i : 0)];
    if (fill) k_guards<true><<<n, GUARD_BYTES / 4, 0, st>>>(g, status);
    else k_guards<false><<<n, GUARD_BYTES / 4, 0, st>>>(g, status);
  }
}

}  // namespace mixaq
