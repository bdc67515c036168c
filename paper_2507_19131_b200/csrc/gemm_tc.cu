// Integer GEMM on the 5th-generation tensor cores (tcgen05.mma kind::i8, u8 activations x s8 weights,
// int32 accumulators in tensor memory) with the fused epilogues of gemm_epilogue.cuh.
//
//   D[128 x BN] (TMEM) = A[128 x K] (u8, K-major, shared memory) * W[BN x K]^T (s8, K-major, shared memory)
//
// Operand staging: 128-byte-swizzled K-major tiles of 128 codes per row and stage.
//   - weights and 8-bit activations arrive by TMA (cp.async.bulk.tensor, no multicast), completion on an mbarrier;
//   - 4-bit / 2-bit activations are read bit-packed from global memory by the producer warps, unpacked to
//     one code per byte in registers and written straight into the swizzled layout the MMA descriptor expects.
// One CTA computes one 128 x BN output tile; several CTAs share an SM so that the epilogue of one overlaps the
// loads and MMAs of another.  Every wait on an mbarrier is bounded; on expiry the CTA raises the status word,
// drains, frees its tensor memory and returns.
#include <cuda.h>
#include "gemm_epilogue.cuh"

namespace mixaq {

namespace {

constexpr int BM = 128;            // rows per tile = TMEM lanes
constexpr int BK = 128;            // codes (bytes) per row and stage = one 128-byte swizzle row
constexpr int UMMA_K = 32;         // codes per tcgen05.mma kind::i8
constexpr int A_STAGE_BYTES = BM * BK;
constexpr int NUM_THREADS = 256;
constexpr int NUM_PRODUCER_WARPS = 6;          // warps 2..7 unpack sub-byte activations
constexpr uint32_t MAX_POLLS = 1u << 22;

struct TcParams {
  GemmArgs g;
  int tiles_m0;          // 128-row tiles of the first (high) branch
  int n_tiles, BN, k_stages, ring, tmem_cols;
  int* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the limit ran out or another thread of the CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < MAX_POLLS; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// shared-memory matrix descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                    // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset
  d |= (uint64_t)1 << 46;                    // descriptor version
  d |= (uint64_t)2 << 61;                    // SWIZZLE_128B
  return d;
}

__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, int32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

template <int MODE>
__global__ void __launch_bounds__(NUM_THREADS)
k_gemm_tc(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
          const __grid_constant__ CUtensorMap tmB, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;                 // swizzled tiles need 1024-byte alignment
  uint8_t* smem = smem_raw + (base - raw);
  const int b_stage_bytes = p.BN * BK;
  const int stage_bytes = A_STAGE_BYTES + b_stage_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)p.ring * stage_bytes);
  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8u * p.ring, bar_acc = bar_empty + 8u * p.ring;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * p.ring + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nt = blockIdx.x % p.n_tiles;
  int mt = blockIdx.x / p.n_tiles;
  const bool is_hi = mt < p.tiles_m0;
  if (!is_hi) mt -= p.tiles_m0;
  const GemmBranch& br = is_hi ? p.g.br[0] : p.g.br[1];
  const CUtensorMap* tmA = is_hi ? &tmA0 : &tmA1;
  const bool packed = br.a_bits != 8;
  const int K = p.g.K;
  const int m0 = mt * BM, n0 = nt * p.BN;

  if (tid == 0) {
    for (int s = 0; s < p.ring; ++s) {
      mbar_init(bar_full + 8u * s, packed ? 1u + NUM_PRODUCER_WARPS : 1u);
      mbar_init(bar_empty + 8u * s, 1u);
    }
    mbar_init(bar_acc, 1u);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_holder)), "r"((uint32_t)p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // ---- TMA producer: weights always, activations when they are stored one code per byte ----
    if (lane == 0) {
      const uint32_t tx = (uint32_t)b_stage_bytes + (packed ? 0u : (uint32_t)A_STAGE_BYTES);
      for (int ks = 0; ks < p.k_stages; ++ks) {
        const int s = ks % p.ring;
        if (ks >= p.ring && !mbar_wait(bar_empty + 8u * s, ((ks / p.ring) - 1) & 1, abort_flag)) break;
        const uint32_t sa = base + (uint32_t)s * stage_bytes, sb = sa + A_STAGE_BYTES;
        mbar_arrive_expect_tx(bar_full + 8u * s, tx);
        tma_load_2d(sb, &tmB, ks * BK, n0, bar_full + 8u * s);
        if (!packed) tma_load_2d(sa, tmA, ks * BK, m0, bar_full + 8u * s);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- MMA issuer: one thread feeds the tensor core ----
    if (lane == 0) {
      const uint32_t idesc = (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(p.BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      bool ok = true;
      for (int ks = 0; ks < p.k_stages && ok; ++ks) {
        const int s = ks % p.ring;
        ok = mbar_wait(bar_full + 8u * s, (ks / p.ring) & 1, abort_flag);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sa = base + (uint32_t)s * stage_bytes, sb = sa + A_STAGE_BYTES;
        const uint64_t adesc = smem_desc_sw128(sa), bdesc = smem_desc_sw128(sb);
        const int ksteps = min(BK, K - ks * BK) / UMMA_K;
        for (int kk = 0; kk < ksteps; ++kk)
          mma_i8(tmem_base, adesc + (uint64_t)(kk * (UMMA_K >> 4)), bdesc + (uint64_t)(kk * (UMMA_K >> 4)), idesc,
                 (ks > 0 || kk > 0) ? 1u : 0u);
        mma_commit(bar_empty + 8u * s);          // frees the ring slot when these MMAs have read it
      }
      if (ok) mma_commit(bar_acc);               // accumulator complete
    }
    __syncwarp();
  } else if (packed) {
    // ---- unpack producers: bit-packed rows -> one code per byte, written in the swizzled layout ----
    const int ptid = tid - 64;                   // 0..191
    const int abits = br.a_bits;
    const long row_bytes = (long)K * abits / 8;
    for (int ks = 0; ks < p.k_stages; ++ks) {
      const int s = ks % p.ring;
      if (ks >= p.ring && !mbar_wait(bar_empty + 8u * s, ((ks / p.ring) - 1) & 1, abort_flag)) break;
      uint8_t* sa = smem + (size_t)s * stage_bytes;
      const int kgroups = min(BK, K - ks * BK) / UMMA_K;       // 32-code groups in this stage
      for (int item = ptid; item < BM * kgroups; item += NUM_PRODUCER_WARPS * 32) {
        const int r = item / kgroups, kg = item - r * kgroups;
        const long m = (long)m0 + r;
        if (m < br.M) {
          uint32_t w[8];
          load_codes_32(br.a + m * row_bytes + (long)(ks * BK + kg * UMMA_K) * abits / 8, abits, w);
          uint8_t* rowp = sa + (r >> 3) * 1024 + (r & 7) * 128;
          const int c0 = (2 * kg) ^ (r & 7), c1 = (2 * kg + 1) ^ (r & 7);
          *reinterpret_cast<uint4*>(rowp + c0 * 16) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(rowp + c1 * 16) = make_uint4(w[4], w[5], w[6], w[7]);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make the writes visible to the MMA proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_full + 8u * s);
    }
    __syncwarp();
  }

  // ---- epilogue: all 8 warps; warp w reads TMEM lanes 32*(w%4).., column groups w/4, w/4+2, ... ----
  const bool acc_ok = mbar_wait(bar_acc, 0, abort_flag);
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (acc_ok) {
    const int q = warp & 3;
    const long m = (long)m0 + q * 32 + lane;
    for (int grp = warp >> 2; grp < p.BN / 32; grp += 2) {
      int32_t acc[32];
      tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(grp * 32), acc);
      if (m < br.M) epilogue_row32<MODE>(br, p.g.N, p.g.C, m, n0 + grp * 32, acc);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (*abort_flag) {
    // a wait ran out: report, and give copies already in flight a bounded chance to land before the CTA exits
    if (tid == 0) {
      atomicExch(p.status, 1);
      for (int s = 0; s < p.ring; ++s)
        for (uint32_t it = 0; it < (1u << 16); ++it)
          if (mbar_try_wait(bar_full + 8u * s, 0) || mbar_try_wait(bar_full + 8u * s, 1)) break;
    }
    __syncthreads();
  }
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
  }
}

// ---- host side -------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// 2-D byte matrix [rows][K] (K contiguous), box = box_rows x 128 bytes, 128-byte swizzle, zero fill outside
bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t K, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {K, rows};
  cuuint64_t strides[1] = {K};
  cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int pick_bn(int N) {
  // the widest tile <= 256 that divides N and is a multiple of 32 (epilogue groups) -- and of 16 (MMA N)
  for (int bn = 256; bn >= 32; bn -= 32)
    if (N % bn == 0) return bn;
  return 0;
}

template <int MODE>
bool launch_mode(const GemmArgs& g, int* status, cudaStream_t st) {
  TcParams p;
  p.g = g; p.status = status;
  const int t0 = (g.br[0].M + BM - 1) / BM, t1 = (g.br[1].M + BM - 1) / BM;
  if (t0 + t1 == 0) return true;
  p.tiles_m0 = t0;
  p.BN = pick_bn(g.N);
  if (p.BN == 0 || g.K % UMMA_K) return false;
  p.n_tiles = g.N / p.BN;
  p.k_stages = (g.K + BK - 1) / BK;
  p.ring = p.k_stages < 4 ? p.k_stages : 4;
  const int stage_bytes = A_STAGE_BYTES + p.BN * BK;
  while (p.ring > 1 && p.ring * stage_bytes > 200 * 1024) --p.ring;
  p.tmem_cols = p.BN <= 32 ? 32 : (p.BN <= 64 ? 64 : (p.BN <= 128 ? 128 : 256));
  CUtensorMap mA[2], mB;
  memset(mA, 0, sizeof(mA));
  for (int i = 0; i < 2; ++i) {
    // branches with packed activations, or without rows, get a valid dummy map of the weights (never used)
    const bool use = g.br[i].M > 0 && g.br[i].a_bits == 8;
    if (!make_map(&mA[i], use ? (const void*)g.br[i].a : (const void*)g.w, use ? (uint64_t)g.br[i].M : (uint64_t)g.N,
                  (uint64_t)g.K, use ? BM : (uint32_t)p.BN))
      return false;
  }
  if (!make_map(&mB, g.w, (uint64_t)g.N, (uint64_t)g.K, (uint32_t)p.BN)) return false;
  const size_t smem = (size_t)p.ring * stage_bytes + 1024 /*alignment slack*/ + (2 * p.ring + 1) * 8 + 16;
  static bool attr_set = false;
  if (!attr_set) {
    cudaFuncSetAttribute(k_gemm_tc<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    attr_set = true;
  }
  k_gemm_tc<MODE><<<(t0 + t1) * p.n_tiles, NUM_THREADS, smem, st>>>(mA[0], mA[1], mB, p);
  ++g_launches;
  return true;
}

}  // namespace

bool launch_gemm_tc(const GemmArgs& g, int* status, cudaStream_t st) {
  switch (g.mode) {
    case EPI_QKV:   return launch_mode<EPI_QKV>(g, status, st);
    case EPI_PROJ:  return launch_mode<EPI_PROJ>(g, status, st);
    case EPI_FC1:   return launch_mode<EPI_FC1>(g, status, st);
    case EPI_FC2:   return launch_mode<EPI_FC2>(g, status, st);
    case EPI_MERGE: return launch_mode<EPI_MERGE>(g, status, st);
  }
  return false;
}

}  // namespace mixaq

namespace mixaq {
bool launch_gemm(const GemmArgs& g, cudaStream_t st) { return launch_gemm_tc(g, g.status, st); }
}  // namespace mixaq
