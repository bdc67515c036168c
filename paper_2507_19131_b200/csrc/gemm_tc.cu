// Integer GEMM on the 5th-generation tensor cores (tcgen05.mma kind::i8, u8 activations x s8 weights,
// int32 accumulators in tensor memory) with the fused epilogues of gemm_epilogue.cuh.
//
//   D[128 x BN] (TMEM) = A[128 x K] (u8, K-major, shared memory) * W[BN x K]^T (s8, K-major, shared memory)
//
// Persistent, warp-specialised: one CTA per SM walks over the output tiles t = blockIdx.x, + gridDim.x, ...
//   warp 0      TMA producer: weight tile and (8-bit branches) activation tile of every k-block into a ring of
//               128-byte-swizzled K-major stages (cp.async.bulk.tensor, no multicast), completion on mbarriers;
//   warp 1      MMA issuer: one thread feeds the tensor core; the accumulator alternates between two TMEM
//               buffers so that the epilogue of tile i overlaps the loads and MMAs of tile i+1;
//   warps 2-5   unpack producers for 4-bit / 2-bit branches: the bit-packed rows of the k-block arrive by TMA in a
//               staging slot of the stage; these warps expand them to one code per byte, shared to shared, into
//               the swizzled layout (rows whose byte pitch is no multiple of 16 cannot be described to the TMA
//               unit and are read with plain loads instead);
//   then        epilogue (12 warps for the code outputs, 8 for the binary32 outputs): tcgen05.ld (one row per thread, 16 columns per load) + the fused epilogue of the mode.
// Every wait on an mbarrier is bounded; on expiry the CTA raises the status word, then waits (bounded again) for the
// copies it has issued to land and for the MMAs it has issued to retire, frees its tensor memory and returns.
#include <cuda.h>
#include "gemm_epilogue.cuh"

namespace mixaq {

namespace {

constexpr int BM = 128;            // rows per tile = TMEM lanes
constexpr int BK = 128;            // codes (bytes) per row and stage = one 128-byte swizzle row
constexpr int UMMA_K = 32;         // codes per tcgen05.mma kind::i8
constexpr int A_STAGE_BYTES = BM * BK;
// warps 2..5 expand sub-byte codes (two warps left the long-K main loops of 4-bit tiles waiting for the expansion;
// eight cost more registers than they return)
__host__ __device__ constexpr int unpack_warps(int mode) { return 4; }
// epilogue warps: 12 for the arithmetic-bound code epilogues, 8 for the binary32 ones
__host__ __device__ constexpr int epi_warps(int mode) { return (mode == EPI_QKV || mode == EPI_FC1) ? 12 : 8; }
constexpr int MAX_BN = 256;
constexpr int EPI_WARP_COLS = MAX_BN / 2;      // most columns one epilogue warp handles per tile (two warps per lane quarter)
constexpr int MAX_RING = 6;
constexpr uint32_t MAX_POLLS = 1u << 22;       // tries per wait

struct TcParams {
  GemmArgs g;
  int tiles_m0;          // 128-row tiles of the first (high) branch
  int total_tiles, n_tiles, BN, k_blocks, ring, tmem_cols;
  int packed_bytes;      // bytes of the packed staging slot of a stage (0: no branch stages packed rows by TMA)
  int res_bytes;         // bytes of the residual rings (proj, fc2: RES_SLOTS chunks per epilogue warp; else 0)
  int tma_packed[2];     // branch i stages its bit-packed rows by TMA (tmA_i then describes the packed matrix)
  int* status;
};

// shared-memory carve-up (offsets from the 1024-byte aligned base)
struct SmemLayout {
  int stage_bytes, ring_bytes, consts_off, stage_off, res_off, bars_off, total;
};
__host__ __device__ inline SmemLayout smem_layout(int BN, int ring, int packed_bytes, int res_bytes, int NUM_EPI_WARPS) {
  SmemLayout L;
  L.stage_bytes = A_STAGE_BYTES + BN * BK + packed_bytes;
  L.ring_bytes = ring * L.stage_bytes;
  L.consts_off = L.ring_bytes;                                  // per epilogue warp (zc, mult, bias) x 128 columns
  L.stage_off = L.consts_off + NUM_EPI_WARPS * 3 * EPI_WARP_COLS * 4;   // per epilogue warp 32 x 16 floats
  L.res_off = L.stage_off + NUM_EPI_WARPS * EPI_STAGE_FLOATS * 4;       // residual rings of the binary32 epilogues
  L.bars_off = L.res_off + res_bytes;
  L.total = L.bars_off + (3 * MAX_RING + 5) * 8 + 16;   // + the drain barrier; then TMEM base, abort flag, fill count
  return L;
}

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
// One try (the hardware suspends the thread for a short, implementation-defined time while the phase is pending;
// an explicit longer suspend hint measured slower: the waiters sit on the critical path of the small stages).
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
struct TileCoord { int mt, nt; bool is_hi; };
__device__ __forceinline__ TileCoord decode_tile(const TcParams& p, int t) {
  TileCoord c;
  c.nt = t % p.n_tiles;
  c.mt = t / p.n_tiles;
  c.is_hi = c.mt < p.tiles_m0;
  if (!c.is_hi) c.mt -= p.tiles_m0;
  return c;
}

// TAPS: the accumulator tap is compiled in only for calls that ask for it
template <int MODE, bool TAPS>
__global__ void __launch_bounds__(32 * (2 + unpack_warps(MODE) + epi_warps(MODE)), 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
          const __grid_constant__ CUtensorMap tmB, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;                 // swizzled tiles need 1024-byte alignment
  uint8_t* smem = smem_raw + (base - raw);
  const SmemLayout L = smem_layout(p.BN, p.ring, p.packed_bytes, p.res_bytes, epi_warps(MODE));
  const int stage_bytes = L.stage_bytes;
  int32_t* s_consts = reinterpret_cast<int32_t*>(smem + L.consts_off);
  float* s_stage = reinterpret_cast<float*>(smem + L.stage_off);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L.bars_off);
  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8u * MAX_RING, bar_raw = bar_empty + 8u * MAX_RING;
  const uint32_t bar_tfull = bar_raw + 8u * MAX_RING, bar_tempty = bar_tfull + 16u, bar_drain = bar_tempty + 16u;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 3 * MAX_RING + 5);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  volatile int* fills_issued = reinterpret_cast<volatile int*>(tmem_holder + 2);   // k-blocks the TMA thread has issued
  int my_arrivals = 0;                       // unpack warps: k-blocks this warp has arrived for on the full barriers

  constexpr int NUM_EPI_WARPS = epi_warps(MODE);
  constexpr int NUM_UNPACK_WARPS = unpack_warps(MODE), NUM_UNPACK_THREADS = NUM_UNPACK_WARPS * 32;
  constexpr int FIRST_EPI_WARP = 2 + NUM_UNPACK_WARPS;
  constexpr int UNPACK_ITEMS = BM * (BK / UMMA_K) / NUM_UNPACK_THREADS;   // (row, 32-code group) items per thread and stage
  constexpr int EPI_SPLIT = NUM_EPI_WARPS / 4;   // warps that share a TMEM lane quarter deal its chunks round-robin
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int K = p.g.K;
  const int acc_stride = p.tmem_cols >> 1;                     // TMEM columns between the two accumulators

  if (tid == 32) {
    // the descriptors are fetched while the barriers are set up
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA0) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA1) : "memory");
  }
  if (tid == 0) {
    for (int s = 0; s < p.ring; ++s) {
      mbar_init(bar_full + 8u * s, 1u + NUM_UNPACK_WARPS);      // TMA thread + one arrival per unpack warp
      mbar_init(bar_empty + 8u * s, 1u);                        // tcgen05.commit
      mbar_init(bar_raw + 8u * s, 1u);                          // TMA thread: "the unpack warps may touch stage s"
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8u * a, 1u);                        // tcgen05.commit of the tile's last MMA
      mbar_init(bar_tempty + 8u * a, NUM_EPI_WARPS);            // one arrival per epilogue warp
    }
    mbar_init(bar_drain, 1u);                                   // tcgen05.commit of the give-up path
    *abort_flag = 0;
    *fills_issued = 0;
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
    // ---- TMA producer ----
    if (lane == 0) {
      int it = 0;                                               // running k-block counter over all tiles of this CTA
      bool ok = true;
      for (int t = blockIdx.x; t < p.total_tiles && ok; t += gridDim.x) {
        const TileCoord tc = decode_tile(p, t);
        const GemmBranch& br = tc.is_hi ? p.g.br[0] : p.g.br[1];
        const bool packed = br.a_bits != 8;
        const bool stage_packed = packed && p.tma_packed[tc.is_hi ? 0 : 1];
        const CUtensorMap* tmA = tc.is_hi ? &tmA0 : &tmA1;
        const uint32_t tx = (uint32_t)(p.BN * BK) + (packed ? 0u : (uint32_t)A_STAGE_BYTES);
        const int pk_row = BK * br.a_bits / 8;                  // packed bytes per row and k-block
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % p.ring;
          if (it >= p.ring && !mbar_wait(bar_empty + 8u * s, ((it / p.ring) - 1) & 1, abort_flag)) { ok = false; break; }
          const uint32_t sa = base + (uint32_t)s * stage_bytes, sb = sa + A_STAGE_BYTES, sp = sb + (uint32_t)(p.BN * BK);
          mbar_arrive_expect_tx(bar_full + 8u * s, tx);
          tma_load_2d(sb, &tmB, kb * BK, tc.nt * p.BN, bar_full + 8u * s);
          if (!packed) tma_load_2d(sa, tmA, kb * BK, tc.mt * BM, bar_full + 8u * s);
          if (stage_packed) {
            mbar_arrive_expect_tx(bar_raw + 8u * s, (uint32_t)(pk_row * BM));
            tma_load_2d(sp, tmA, kb * pk_row, tc.mt * BM, bar_raw + 8u * s);
          } else {
            mbar_arrive(bar_raw + 8u * s);
          }
        }
      }
      *fills_issued = it;                                       // read by the give-up path only
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- MMA issuer ----
    if (lane == 0) {
      const uint32_t idesc = (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(p.BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      int it = 0, lt = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < p.total_tiles && ok; t += gridDim.x, ++lt) {
        const int a = lt & 1;
        // wait until the epilogue has drained this accumulator (its use two tiles ago)
        if (lt >= 2 && !mbar_wait(bar_tempty + 8u * a, ((lt >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + (uint32_t)(a * acc_stride);
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % p.ring;
          if (!mbar_wait(bar_full + 8u * s, (it / p.ring) & 1, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sa = base + (uint32_t)s * stage_bytes, sb = sa + A_STAGE_BYTES;
          const uint64_t adesc = smem_desc_sw128(sa), bdesc = smem_desc_sw128(sb);
          const int ksteps = min(BK, K - kb * BK) / UMMA_K;
          for (int kk = 0; kk < ksteps; ++kk)
            mma_i8(d_tmem, adesc + (uint64_t)(kk * (UMMA_K >> 4)), bdesc + (uint64_t)(kk * (UMMA_K >> 4)), idesc,
                   (kb > 0 || kk > 0) ? 1u : 0u);
          mma_commit(bar_empty + 8u * s);          // frees the ring slot when these MMAs have read it
        }
        if (ok) mma_commit(bar_tfull + 8u * a);    // accumulator complete
      }
    }
    __syncwarp();
  } else if (warp < FIRST_EPI_WARP) {
    // ---- unpack producers: bit-packed rows -> one code per byte, written in the swizzled layout ----
    const int ptid = tid - 64;                   // 0 .. NUM_UNPACK_THREADS-1
    int it = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < p.total_tiles && ok; t += gridDim.x) {
      const TileCoord tc = decode_tile(p, t);
      const GemmBranch& br = tc.is_hi ? p.g.br[0] : p.g.br[1];
      const int abits = br.a_bits;
      const bool packed = abits != 8;
      const bool staged = packed && p.tma_packed[tc.is_hi ? 0 : 1];
      const long row_bytes = (long)K * abits / 8;
      const long m0 = (long)tc.mt * BM;
      const int grp_bytes = UMMA_K * abits / 8;                 // packed bytes of one 32-code group
      for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
        const int s = it % p.ring;
        // the TMA thread arrives on raw[s] once it owns the stage (and, when staged, the packed bytes have landed)
        if (!mbar_wait(bar_raw + 8u * s, (it / p.ring) & 1, abort_flag)) { ok = false; break; }
        if (packed) {
          uint8_t* sa = smem + (size_t)s * stage_bytes;
          const uint8_t* sp = sa + A_STAGE_BYTES + p.BN * BK;
          const int kgroups = min(BK, K - kb * BK) / UMMA_K;
          // item i of this thread: row r = item / 4, 32-code group kg = item % 4, item = ptid + NUM_UNPACK_THREADS * i
#pragma unroll
          for (int i = 0; i < UNPACK_ITEMS; ++i) {
            const int item = ptid + NUM_UNPACK_THREADS * i;
            const int r = item >> 2, kg = item & 3;
            uint32_t w[8];
            bool have = true;
            if (staged) {
              // rows and columns outside the matrix were zero-filled by the TMA unit
              load_codes_32(sp + item * grp_bytes, abits, w);
            } else {
              have = kg < kgroups && m0 + r < br.M;
              if (have) load_codes_32(br.a + (m0 + r) * row_bytes + (long)(kb * BK + kg * UMMA_K) * abits / 8, abits, w);
            }
            if (have) {
              uint8_t* rowp = sa + (r >> 3) * 1024 + (r & 7) * 128;
              const int c0 = (2 * kg) ^ (r & 7), c1 = (2 * kg + 1) ^ (r & 7);
              *reinterpret_cast<uint4*>(rowp + c0 * 16) = make_uint4(w[0], w[1], w[2], w[3]);
              *reinterpret_cast<uint4*>(rowp + c1 * 16) = make_uint4(w[4], w[5], w[6], w[7]);
            }
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make the writes visible to the MMA proxy
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_full + 8u * s);
      }
    }
    my_arrivals = it;
    __syncwarp();
  } else {
    // ---- epilogue warps: warp e reads TMEM lanes 32*(e%4).. and takes every EPI_SPLIT-th 16-column chunk ----
    const int e = warp - FIRST_EPI_WARP, q = warp & 3, sub = e >> 2;   // any 4 consecutive warps cover the 4 lane quarters
    float* stage = s_stage + e * EPI_STAGE_FLOATS;
    float* res_ring = reinterpret_cast<float*>(smem + L.res_off) + e * RES_SLOTS * EPI_STAGE_FLOATS;
    int32_t* c_zc = s_consts + e * 3 * EPI_WARP_COLS;
    float* c_mult = reinterpret_cast<float*>(c_zc + EPI_WARP_COLS);
    float* c_bias = c_mult + EPI_WARP_COLS;
    const int c_total = p.BN / EPI_NC;                         // BN is a multiple of 32
    int lt = 0, consts_key = -1;
    // the tile walk without a division per tile: (row tile, column tile) advance by gridDim.x tiles at a time
    const int step_m = (int)gridDim.x / p.n_tiles, step_n = (int)gridDim.x % p.n_tiles;
    int w_mt = (int)blockIdx.x / p.n_tiles, w_nt = (int)blockIdx.x % p.n_tiles;
    for (int t = blockIdx.x; t < p.total_tiles; t += gridDim.x, ++lt) {
      TileCoord tc;
      tc.nt = w_nt; tc.mt = w_mt; tc.is_hi = w_mt < p.tiles_m0;
      if (!tc.is_hi) tc.mt -= p.tiles_m0;
      w_mt += step_m; w_nt += step_n;
      if (w_nt >= p.n_tiles) { w_nt -= p.n_tiles; ++w_mt; }
      const GemmBranch& br = tc.is_hi ? p.g.br[0] : p.g.br[1];
      const int a = lt & 1;
      const int n_tile0 = tc.nt * p.BN;
      // per-column constants of this warp's chunks, densely in the warp's own shared-memory slot; they depend on
      // the branch and the column tile only, and the grid is sized so that a CTA keeps its column tile
      // (no CTA-wide barrier: the only waits of this kernel are the bounded mbarrier waits)
      const int key = tc.nt * 2 + (tc.is_hi ? 1 : 0);
      if (key != consts_key) {
        consts_key = key;
        __syncwarp();
        for (int c = sub, j = 0; c < c_total; c += EPI_SPLIT, ++j) {
          if (lane < EPI_NC) {
            const int n = n_tile0 + c * EPI_NC + lane;
            c_zc[j * EPI_NC + lane] = __ldg(br.zc + n);
            c_mult[j * EPI_NC + lane] = __ldg(br.mult + n);
            if (MODE != EPI_MERGE) c_bias[j * EPI_NC + lane] = __ldg(br.bias + n);
          }
        }
        __syncwarp();
      }
      ColConsts cc; cc.zc = c_zc; cc.mult = c_mult; cc.bias = c_bias;
      const long row0 = (long)tc.mt * BM + q * 32;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * acc_stride);
      auto acc_ready = [&]() -> bool {
        if (!mbar_wait(bar_tfull + 8u * a, (lt >> 1) & 1, abort_flag)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        return true;
      };
      if (!epilogue_warp_tile<MODE, TAPS>(br, p.g.N, p.g.C, row0, lane, n_tile0, sub, EPI_SPLIT, c_total, cc, taddr, stage,
                                    acc_ready, res_ring)) break;
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8u * a);
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (*abort_flag) {
    // A wait ran out.  Before the CTA may exit, the copies already issued must have landed in its shared memory and
    // the MMAs already issued must have retired.  (1) Every unpack warp arrives, on the full barrier of each k-block
    // that was issued but that it had not reached, so that those phases can complete once their bytes are there
    // (the ring admits at most one such k-block per stage).  (2) The MMA thread commits what it has issued to a
    // barrier of its own.  (3) One thread waits, bounded, for the phase of the LAST fill of every stage, on the
    // packed-rows barrier and on the full barrier, and for the MMA commit.
    const int issued = *fills_issued;
    if (warp >= 2 && warp < FIRST_EPI_WARP && lane == 0)
      for (int j = my_arrivals; j < issued; ++j) mbar_arrive(bar_full + 8u * (uint32_t)(j % p.ring));
    if (tid == 32) mma_commit(bar_drain);
    __syncthreads();
    if (tid == 0) {
      atomicExch(p.status, 1);
      auto drain = [](uint32_t bar, uint32_t parity) {
        for (uint32_t it = 0; it < (1u << 20); ++it) if (mbar_try_wait(bar, parity)) return;
      };
      for (int s = 0; s < p.ring; ++s) {
        const int fills = issued > s ? (issued - s + p.ring - 1) / p.ring : 0;     // k-blocks j < issued with j % ring == s
        if (fills == 0) continue;
        const uint32_t parity = (uint32_t)(fills - 1) & 1u;
        drain(bar_raw + 8u * s, parity);
        drain(bar_full + 8u * s, parity);
      }
      drain(bar_drain, 0u);
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

// 2-D byte matrix [rows][row_bytes] (bytes of a row contiguous), box = box_rows x box_bytes, zero fill outside.
// swizzled: 128-byte swizzle for MMA operand tiles (box_bytes = 128); otherwise a plain row-major box.
bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t row_bytes, uint32_t box_rows,
              uint32_t box_bytes = BK, bool swizzled = true) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {row_bytes, rows};
  cuuint64_t strides[1] = {row_bytes};
  cuuint32_t box[2] = {box_bytes, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzled ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int num_sms() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
  }
  return n;
}

// Tile width: a multiple of 32 (epilogue groups) that divides N, at most 256; among those, the one that needs the
// fewest "waves x (columns per tile + fixed per-tile work)" on this many SMs.
int pick_bn(int N, int m_tiles, int sms) {
  int best = 0; long best_cost = 0;
  for (int bn = 32; bn <= MAX_BN; bn += 32) {
    if (N % bn) continue;
    const long tiles = (long)m_tiles * (N / bn);
    const long waves = (tiles + sms - 1) / sms;
    const long cost = waves * (bn + 48);
    if (!best || cost <= best_cost) { best = bn; best_cost = cost; }
  }
  return best;
}

template <int MODE>
bool launch_mode(const GemmArgs& g, int* status, cudaStream_t st) {
  TcParams p;
  p.g = g; p.status = status;
  const int t0 = (g.br[0].M + BM - 1) / BM, t1 = (g.br[1].M + BM - 1) / BM;
  if (t0 + t1 == 0) return true;
  if (g.N % 32 || g.K % UMMA_K) return false;
  const int sms = num_sms();
  p.tiles_m0 = t0;
  p.BN = pick_bn(g.N, t0 + t1, sms);
  if (p.BN == 0) return false;
  p.n_tiles = g.N / p.BN;
  p.total_tiles = (t0 + t1) * p.n_tiles;
  p.k_blocks = (g.K + BK - 1) / BK;
  // packed branches whose row pitch the TMA unit accepts (a multiple of 16 bytes) are staged by TMA
  p.packed_bytes = 0;
  for (int i = 0; i < 2; ++i) {
    const int bits = g.br[i].a_bits;
    p.tma_packed[i] = g.br[i].M > 0 && bits != 8 && ((long)g.K * bits / 8) % 16 == 0;
    if (p.tma_packed[i]) p.packed_bytes = BM * (BK / 2);        // room for the widest packed format (4 bit)
  }
  p.res_bytes = (g.mode == EPI_PROJ || g.mode == EPI_FC2) ? epi_warps(g.mode) * RES_SLOTS * EPI_STAGE_FLOATS * 4 : 0;
  p.ring = MAX_RING;
  while (p.ring > 2 && smem_layout(p.BN, p.ring, p.packed_bytes, p.res_bytes, epi_warps(MODE)).total + 1024 > 220 * 1024) --p.ring;
  p.tmem_cols = 32;
  while (p.tmem_cols < 2 * p.BN) p.tmem_cols <<= 1;
  CUtensorMap mA[2], mB;
  memset(mA, 0, sizeof(mA));
  for (int i = 0; i < 2; ++i) {
    const GemmBranch& b = g.br[i];
    bool ok;
    if (b.M > 0 && b.a_bits == 8)
      ok = make_map(&mA[i], b.a, (uint64_t)b.M, (uint64_t)g.K, BM);
    else if (p.tma_packed[i])
      ok = make_map(&mA[i], b.a, (uint64_t)b.M, (uint64_t)g.K * b.a_bits / 8, BM, (uint32_t)(BK * b.a_bits / 8), false);
    else   // no rows, or rows read with plain loads: a valid map of the weights that is never used
      ok = make_map(&mA[i], g.w, (uint64_t)g.N, (uint64_t)g.K, (uint32_t)p.BN);
    if (!ok) return false;
  }
  if (!make_map(&mB, g.w, (uint64_t)g.N, (uint64_t)g.K, (uint32_t)p.BN)) return false;
  const size_t smem = (size_t)smem_layout(p.BN, p.ring, p.packed_bytes, p.res_bytes, epi_warps(MODE)).total + 1024 /*alignment slack*/;
  if (smem > 227 * 1024) return false;
  // a grid that is a multiple of the number of column tiles keeps every CTA on one column tile (t mod n_tiles);
  // taken only where it does not cost a wave of tiles
  int grid = p.total_tiles < sms ? p.total_tiles : sms;
  if (grid > p.n_tiles && grid < p.total_tiles) {
    const int g2 = grid - grid % p.n_tiles;
    if ((p.total_tiles + g2 - 1) / g2 == (p.total_tiles + grid - 1) / grid) grid = g2;
  }
  if (g.br[0].tap_acc || g.br[1].tap_acc)
    k_gemm_tc<MODE, true><<<grid, 32 * (2 + unpack_warps(MODE) + epi_warps(MODE)), smem, st>>>(mA[0], mA[1], mB, p);
  else
    k_gemm_tc<MODE, false><<<grid, 32 * (2 + unpack_warps(MODE) + epi_warps(MODE)), smem, st>>>(mA[0], mA[1], mB, p);
  ++g_launches;
  return true;
}

}  // namespace

// The bounded wait of this file on a barrier that nothing ever signals: it has to run out, raise the status word and
// let the CTA return normally.  (One CTA, one thread; no copy and no tensor memory is involved.)
__global__ void k_wait_probe(int* status, uint32_t tries) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    bool done = false;
    for (uint32_t it = 0; it < tries && !done; ++it) done = mbar_try_wait(smem_u32(&bar), 0);
    if (!done) atomicExch(status, 1);
  }
}

void launch_wait_probe(int* status, cudaStream_t st) {
  k_wait_probe<<<1, 32, 0, st>>>(status, 4096u);    // a few thousand tries: well under a millisecond
  ++g_launches;
}

// Issue-rate microbenchmark of the tensor core: every CTA (one per SM) keeps a 128 x 128-byte A tile and a
// 256 x 128-byte B tile in shared memory and issues `groups` x 4 MMAs of 128 x 256 x 32 into one TMEM accumulator,
// then waits (bounded) for the commit.  KIND 0: kind::i8 (u8 x s8 -> s32), the path the GEMMs use.
// KIND 1: kind::f8f6f4 with E4M3 operands (-> f32); this is also the path that carries 4-bit and 6-bit operand
// formats on sm_100a (in 8-bit shared-memory containers), so its rate bounds what a narrower operand type could give.
// KIND 2: kind::mxf4 (E2M1 operands packed two per byte, one UE8M0 scale per 32 values, -> f32): 128 x 256 x 64 per
// instruction from the same 32 bytes per row, the only narrower path with a higher nominal rate.
template <int KIND>
__global__ void __launch_bounds__(128, 1) k_mma_peak(int groups, unsigned long long* ns_out, int* status) {
  constexpr uint32_t PEAK_TMEM_COLS = KIND == 2 ? 512u : 256u;   // KIND 2 keeps its scale factors behind the accumulator
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  uint64_t* bar = reinterpret_cast<uint64_t*>(smem + A_STAGE_BYTES + MAX_BN * BK);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bar + 1);
  const int tid = threadIdx.x, warp = tid >> 5;
  for (int i = tid; i < (A_STAGE_BYTES + MAX_BN * BK) / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(smem)[i] = ((uint32_t)(i * 37 + 11) * 0x01010101u) & 0x3E3E3E3Eu;   // finite in E4M3 too
  if (tid == 0) { mbar_init(smem_u32(bar), 1u); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)), "r"(PEAK_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_holder;
  if (tid == 0) {
    // instruction descriptor: D format (s32 = 2 / f32 = 1) at bit 4, A format at 7, B format at 10, N/8 at 17, M/16 at 24
    // (block-scaled kinds: no D format field; A and B format 1 = E2M1 at bits 7 and 10, scale format 1 = UE8M0 at bit 23)
    const uint32_t idesc = KIND == 0 ? ((2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(MAX_BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24))
                         : KIND == 1 ? ((1u << 4) | (0u << 7) | (0u << 10) | ((uint32_t)(MAX_BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24))
                                     : ((1u << 7) | (1u << 10) | ((uint32_t)(MAX_BN >> 3) << 17) | (1u << 23) | ((uint32_t)(BM >> 4) << 24));
    // KIND 2: the scale factors of A and B sit in tensor memory behind the accumulator (columns 256.., 264..); their
    // contents are whatever the allocation holds -- the products are meaningless, only the issue rate is measured
    const uint32_t sfa = tmem_base + 256u, sfb = tmem_base + 264u;
    const uint64_t adesc = smem_desc_sw128(base), bdesc = smem_desc_sw128(base + A_STAGE_BYTES);
    unsigned long long t0, t1;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
    for (int g = 0; g < groups; ++g)
      for (int kk = 0; kk < BK / UMMA_K; ++kk) {
        const uint32_t accumulate = (g > 0 || kk > 0) ? 1u : 0u;
        if (KIND == 0) {
          mma_i8(tmem_base, adesc + (uint64_t)(kk * (UMMA_K >> 4)), bdesc + (uint64_t)(kk * (UMMA_K >> 4)), idesc, accumulate);
        } else if (KIND == 2) {
          // 32 bytes of a row are 64 E2M1 values: one MMA of 128 x 256 x 64 with one UE8M0 scale per 32 values
          asm volatile(
              "{\n\t.reg .pred p;\n\t"
              "setp.ne.b32 p, %4, 0;\n\t"
              "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
              ::"r"(tmem_base), "l"(adesc + (uint64_t)(kk * (UMMA_K >> 4))), "l"(bdesc + (uint64_t)(kk * (UMMA_K >> 4))),
                "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb) : "memory");
        } else {
          asm volatile(
              "{\n\t.reg .pred p;\n\t"
              "setp.ne.b32 p, %4, 0;\n\t"
              "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
              ::"r"(tmem_base), "l"(adesc + (uint64_t)(kk * (UMMA_K >> 4))), "l"(bdesc + (uint64_t)(kk * (UMMA_K >> 4))),
                "r"(idesc), "r"(accumulate) : "memory");
        }
      }
    mma_commit(smem_u32(bar));
    bool done = false;
    for (uint32_t it = 0; it < MAX_POLLS && !done; ++it) done = mbar_try_wait(smem_u32(bar), 0);
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
    if (!done) atomicExch(status, 1);
    ns_out[blockIdx.x] = t1 - t0;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(PEAK_TMEM_COLS) : "memory");
}

// ns_out: one entry per SM (device memory).  Returns the grid size, 0 on failure.
int launch_mma_peak(int kind, int groups, unsigned long long* ns_out, int* status, cudaStream_t st) {
  const int sms = num_sms();
  const size_t smem = A_STAGE_BYTES + MAX_BN * BK + 1024 + 64;
  if (kind == 0) {
    if (cudaFuncSetAttribute(k_mma_peak<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 0;
    k_mma_peak<0><<<sms, 128, smem, st>>>(groups, ns_out, status);
  } else if (kind == 1) {
    if (cudaFuncSetAttribute(k_mma_peak<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 0;
    k_mma_peak<1><<<sms, 128, smem, st>>>(groups, ns_out, status);
  } else {
    if (cudaFuncSetAttribute(k_mma_peak<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 0;
    k_mma_peak<2><<<sms, 128, smem, st>>>(groups, ns_out, status);
  }
  ++g_launches;
  return sms;
}

// One-time set-up per device context (kept out of the launch path so that launches can be stream-captured):
// opt-in to large dynamic shared memory for every epilogue mode, resolve the tensor-map encoder, read the SM count.
bool gemm_init() {
  bool ok = encode_fn() != nullptr && num_sms() > 0;
  ok &= cudaFuncSetAttribute(k_gemm_tc<EPI_QKV, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
  ok &= cudaFuncSetAttribute(k_gemm_tc<EPI_QKV, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
  ok &= cudaFuncSetAttribute(k_gemm_tc<EPI_PROJ, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
  ok &= cudaFuncSetAttribute(k_gemm_tc<EPI_PROJ, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
  ok &= cudaFuncSetAttribute(k_gemm_tc<EPI_FC1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
  ok &= cudaFuncSetAttribute(k_gemm_tc<EPI_FC1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
  ok &= cudaFuncSetAttribute(k_gemm_tc<EPI_FC2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
  ok &= cudaFuncSetAttribute(k_gemm_tc<EPI_FC2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
  ok &= cudaFuncSetAttribute(k_gemm_tc<EPI_MERGE, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
  ok &= cudaFuncSetAttribute(k_gemm_tc<EPI_MERGE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
  return ok;
}

bool launch_gemm(const GemmArgs& g, cudaStream_t st) {
  switch (g.mode) {
    case EPI_QKV:   return launch_mode<EPI_QKV>(g, g.status, st);
    case EPI_PROJ:  return launch_mode<EPI_PROJ>(g, g.status, st);
    case EPI_FC1:   return launch_mode<EPI_FC1>(g, g.status, st);
    case EPI_FC2:   return launch_mode<EPI_FC2>(g, g.status, st);
    case EPI_MERGE: return launch_mode<EPI_MERGE>(g, g.status, st);
  }
  return false;
}

}  // namespace mixaq
