// Fused epilogues of the integer GEMMs (MixA-Q Section 3.2: shared integer weights, per-branch step sizes,
// zero points and biases).  One epilogue warp owns 32 rows (one TMEM lane quarter, one row per thread) and every
// c_step-th 16-column chunk of the tile (the warps that share a lane quarter deal the chunks round-robin):
//   acc_raw[n] = sum_k a[m][k] * w[n][k]   with UNSIGNED activation codes a;
//   acc[n]     = acc_raw[n] - z_a * sum_k w[n][k]                (zero-point correction, exact in int32)
//   v[n]       = fma((float)acc[n], s_a*s_w[n], bias[n])
// The per-column constants (zc, mult, bias) of the warp's columns sit in shared memory; every lane reads the same
// column, so the reads are broadcasts.
#pragma once
#include "kernels.h"

namespace mixaq {

constexpr int EPI_NC = 16;                             // columns per chunk
constexpr int EPI_STAGE_FLOATS = 32 * EPI_NC;          // per-warp transposition tile of the binary32 epilogues

struct ColConsts {                                     // shared-memory arrays indexed by the warp's local column
  const int32_t* zc; const float* mult; const float* bias;
};

// Asynchronous TMEM load of 16 columns (one row per thread); the registers are valid after tmem_ld_wait().
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, int32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
// Waits for every TMEM load issued so far.  The registers pass through the statement as in-out operands so that
// no use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait(int32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
      : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
        "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
      :: "memory");
}

// asynchronous 16-byte copy global -> shared (no register staging); groups complete in order
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

constexpr int RES_SLOTS = 4;                           // residual chunks a warp keeps in flight (32 x 16 floats each)

// zero-point correction + dequantization of one chunk; lc0 = first column of the chunk in the warp's constants
template <int MODE, bool TAPS>
__device__ __forceinline__ void dequant16(const GemmBranch& br, int N, long m, bool row_ok, int n0, int lc0,
                                          const ColConsts& cc, const int32_t (&acc_raw)[16], float (&v)[16]) {
  if (TAPS && br.tap_acc && row_ok) {
#pragma unroll
    for (int i = 0; i < EPI_NC; ++i) br.tap_acc[m * N + n0 + i] = acc_raw[i] - cc.zc[lc0 + i];
  }
#pragma unroll
  for (int i4 = 0; i4 < EPI_NC / 4; ++i4) {
    const int4 z4 = *reinterpret_cast<const int4*>(cc.zc + lc0 + 4 * i4);
    const float4 m4 = *reinterpret_cast<const float4*>(cc.mult + lc0 + 4 * i4);
    const int zz[4] = {z4.x, z4.y, z4.z, z4.w};
    const float mm[4] = {m4.x, m4.y, m4.z, m4.w};
    float bb[4] = {0.f, 0.f, 0.f, 0.f};
    if (MODE != EPI_MERGE) {
      const float4 b4 = *reinterpret_cast<const float4*>(cc.bias + lc0 + 4 * i4);
      bb[0] = b4.x; bb[1] = b4.y; bb[2] = b4.z; bb[3] = b4.w;
    }
    // two columns per packed instruction (each lane rounds like the scalar fma / mul)
#pragma unroll
    for (int j = 0; j < 4; j += 2) {
      const int i = 4 * i4 + j;
      const float2 f = make_float2(__int2float_rn(acc_raw[i] - zz[j]), __int2float_rn(acc_raw[i + 1] - zz[j + 1]));
      const float2 r = MODE == EPI_MERGE ? __fmul2_rn(f, make_float2(mm[j], mm[j + 1]))
                                         : __ffma2_rn(f, make_float2(mm[j], mm[j + 1]), make_float2(bb[j], bb[j + 1]));
      v[i] = r.x; v[i + 1] = r.y;
    }
  }
}

// The warp's part of one output tile.  taddr: TMEM address of (the warp's lane quarter, the tile's first column);
// n_tile0: global index of that column; the warp owns the tile's chunks c_first, c_first + c_step, ... < c_total
// (its constants are stored densely: chunk number j of the warp at local column 16 j);
// acc_ready(): waits (bounded) for the tile's accumulator, false when the CTA is giving up.
template <int MODE, bool TAPS, class WaitFn>
__device__ __forceinline__ bool epilogue_warp_tile(const GemmBranch& br, int N, int C, long row0, int lane, int n_tile0,
                                                   int c_first, int c_step, int c_total, const ColConsts& cc,
                                                   uint32_t taddr_tile, float* stage, WaitFn acc_ready,
                                                   float* res_ring = nullptr /* per warp: RES_SLOTS x 32 x 16 floats */) {
  const long m = row0 + lane;
  const bool row_ok = m < br.M;
  const int n_chunks = c_first < c_total ? (c_total - c_first + c_step - 1) / c_step : 0;
  const int n_first = n_tile0 + c_first * EPI_NC;          // global column of the warp's first chunk
  const int col_step = c_step * EPI_NC;                    // distance between consecutive chunks of the warp
  const uint32_t taddr = taddr_tile + (uint32_t)(c_first * EPI_NC);

  if (MODE == EPI_QKV || MODE == EPI_FC1) {
    // ---- code outputs: every thread quantizes and packs the 16 codes of its own row ----
    if (!acc_ready()) return false;
    const int bits = br.out_bits;
    // this thread's output position of the warp's first chunk; packing constants of the (up to three) quantizers
    uint8_t* out_ptr = br.out_codes + m * ((long)N * bits / 8) + (long)n_first * bits / 8;
    const int out_step = col_step * bits / 8;
    const uint32_t kp0 = pack_const(br.q0.zp, bits);
    const uint32_t kp1 = MODE == EPI_QKV ? pack_const(br.q1.zp, bits) : kp0;
    const uint32_t kp2 = MODE == EPI_QKV ? pack_const(br.q2.zp, bits) : kp0;
    const int n_k = C, n_v = 2 * C;                      // first columns of the k and v sections (QKV)
    auto chunk = [&](int ch, const int32_t (&acc)[EPI_NC]) {
      const int n0 = n_first + ch * col_step;
      float v[EPI_NC];
      dequant16<MODE, TAPS>(br, N, m, row_ok, n0, ch * EPI_NC, cc, acc, v);
      AQ q = br.q0;
      uint32_t kp = kp0;
      if (MODE == EPI_QKV) { if (n0 >= n_v) { q = br.q2; kp = kp2; } else if (n0 >= n_k) { q = br.q1; kp = kp1; } }
      uint32_t c[EPI_NC];
      const float q_lo = -q.zpf, q_hi = q.qmaxf - q.zpf;
#pragma unroll
      for (int i = 0; i < EPI_NC; i += 2) {
        float2 g = make_float2(v[i], v[i + 1]);
        if (MODE == EPI_FC1) g = gelu_f2(g);
        quant_magic2(g, q.inv_scale, q_lo, q_hi, c[i], c[i + 1]);
      }
      if (row_ok) {
        uint8_t* dst = out_ptr + ch * out_step;
        if (bits == 8) store_magic<8, EPI_NC>(dst, c, kp);
        else if (bits == 4) store_magic<4, EPI_NC>(dst, c, kp);
        else store_magic<2, EPI_NC>(dst, c, kp);
      }
    };
    // the TMEM load of the next chunk is in flight while this chunk is computed
    // (one copy of the chunk body keeps the loop inside the instruction cache: the prefetched registers are moved)
    int32_t acc[EPI_NC], nxt[EPI_NC];
    if (n_chunks > 0) tmem_ld16_issue(taddr, nxt);
#pragma unroll 1
    for (int ch = 0; ch < n_chunks; ++ch) {
      tmem_ld_wait(nxt);
#pragma unroll
      for (int i = 0; i < EPI_NC; ++i) acc[i] = nxt[i];
      if (ch + 1 < n_chunks) tmem_ld16_issue(taddr + (uint32_t)((ch + 1) * col_step), nxt);
      chunk(ch, acc);
    }
    return true;
  }

  // ---- binary32 outputs (proj: x1 = x_window + out; fc2: y = x1 + out scattered to the token's own position;
  //      merge: out).  Each chunk is transposed through shared memory so that global accesses are 64-byte runs
  //      (4 lanes per row, 8 rows per instruction). ----
  const int cj = lane & 3, rsub = lane >> 2;
  long src_mine = -1;
  if (MODE != EPI_MERGE && row_ok) src_mine = br.rowsrc[m];
  // this lane's four (row, 16-byte piece) positions of the warp's first chunk: residual source and output, NULL: none
  const float* res_ptr[4];
  float* dst_ptr[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = 8 * i + rsub;
    const long mr = row0 + r;
    const long s = __shfl_sync(0xffffffffu, src_mine, r);
    const bool ok = mr < br.M;
    long res_row, dst_row;               // row offsets (in elements), -1: none
    if (MODE == EPI_PROJ)     { res_row = (ok && s >= 0) ? s * N : -1;  dst_row = ok ? mr * N : -1; }
    else if (MODE == EPI_FC2) { res_row = (ok && s >= 0) ? mr * N : -1; dst_row = (ok && s >= 0) ? s * N : -1; }
    else                      { res_row = -1;                            dst_row = ok ? mr * N : -1; }
    res_ptr[i] = (MODE != EPI_MERGE && res_row >= 0) ? br.res + res_row + n_first + 4 * cj : nullptr;
    dst_ptr[i] = dst_row >= 0 ? br.out_f + dst_row + n_first + 4 * cj : nullptr;
  }
  // The residual rows come into shared memory by asynchronous copies, RES_SLOTS chunks ahead of their use: the copies
  // of a whole tile are in flight while the accumulator is still being computed, and they cost no registers.
  // Slot ch % RES_SLOTS holds chunk ch in the layout of the transposition tile (row r, 16-byte piece j at piece
  // j ^ ((r >> 1) & 3)).  One commit group per chunk, also when there is nothing left to fetch, so that "all but the
  // newest RES_SLOTS - 1 groups are complete" always covers the chunk about to be used.
  auto fetch = [&](int ch) {
    if (MODE != EPI_MERGE && ch < n_chunks) {
      float* slot = res_ring + (ch % RES_SLOTS) * EPI_STAGE_FLOATS;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = 8 * i + rsub;
        float* dst = slot + r * EPI_NC + 4 * (cj ^ ((r >> 1) & 3));
        if (res_ptr[i]) cp_async16(dst, res_ptr[i] + ch * col_step);
        else *reinterpret_cast<float4*>(dst) = make_float4(0.f, 0.f, 0.f, 0.f);   // a pad token's residual input is zero
      }
    }
    cp_async_commit();
  };
  if (MODE != EPI_MERGE) {
#pragma unroll
    for (int ch = 0; ch < RES_SLOTS; ++ch) fetch(ch);
  }
  if (!acc_ready()) { cp_async_wait<0>(); return false; }
  auto chunk = [&](int ch, const int32_t (&acc)[EPI_NC]) {
    const int n0 = n_first + ch * col_step;
    float v[EPI_NC];
    dequant16<MODE, TAPS>(br, N, m, row_ok, n0, ch * EPI_NC, cc, acc, v);
    // row `lane`, logical 16-byte piece j is stored at piece j ^ ((lane >> 1) & 3): conflict-free both ways
#pragma unroll
    for (int j = 0; j < 4; ++j)
      *reinterpret_cast<float4*>(stage + lane * EPI_NC + 4 * (j ^ ((lane >> 1) & 3))) =
          make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
    if (MODE != EPI_MERGE) cp_async_wait<RES_SLOTS - 1>();     // this lane's copies of chunk ch have landed
    __syncwarp();
    const float* slot = res_ring + (ch % RES_SLOTS) * EPI_STAGE_FLOATS;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = 8 * i + rsub;
      const int off = r * EPI_NC + 4 * (cj ^ ((r >> 1) & 3));
      const float4 a = *reinterpret_cast<const float4*>(stage + off);
      if (dst_ptr[i]) {
        float4 o = a;
        if (MODE != EPI_MERGE) {
          const float4 rr = *reinterpret_cast<const float4*>(slot + off);
          const float2 lo = __fadd2_rn(make_float2(rr.x, rr.y), make_float2(a.x, a.y));
          const float2 hi = __fadd2_rn(make_float2(rr.z, rr.w), make_float2(a.z, a.w));
          o = make_float4(lo.x, lo.y, hi.x, hi.y);
        }
        *reinterpret_cast<float4*>(dst_ptr[i] + ch * col_step) = o;
      }
    }
    __syncwarp();
    if (MODE != EPI_MERGE) fetch(ch + RES_SLOTS);              // the slot just read is free again
  };
  int32_t acc[EPI_NC], nxt[EPI_NC];
  if (n_chunks > 0) tmem_ld16_issue(taddr, nxt);
#pragma unroll 1
  for (int ch = 0; ch < n_chunks; ++ch) {
    tmem_ld_wait(nxt);
#pragma unroll
    for (int i = 0; i < EPI_NC; ++i) acc[i] = nxt[i];
    if (ch + 1 < n_chunks) tmem_ld16_issue(taddr + (uint32_t)((ch + 1) * col_step), nxt);
    chunk(ch, acc);
  }
  if (MODE != EPI_MERGE) cp_async_wait<0>();                   // nothing of this tile is left in flight
  return true;
}

}  // namespace mixaq
