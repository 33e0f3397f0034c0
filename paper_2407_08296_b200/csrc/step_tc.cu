// Tensor-core version of the Q-GaLore step (Sec. 3.5) for sm_100a: two persistent, warp-specialised
// kernels over a table of matrices ("problems"), both built on tcgen05.mma with the accumulator in
// tensor memory and every operand tile brought in by TMA.
//
//   project_adam_kernel   R = P~^T G  (tile 128 rows of r x BN columns of n, K = m), then per tile the
//                         Adam update of M, V (Kingma & Ba) and the bf16 direction N_b -> workspace.
//   backproject_sr_kernel D = P~ N_b  (tile 128 rows of m x 256 columns of n, K = r), then per tile
//                         W' = dequant(W) - lr*alpha*D - lr*wd*dequant(W) and Quant_8 with stochastic
//                         rounding (Sec. 3.4).  A tile row is exactly one quantization group, and a
//                         thread of the epilogue owns one accumulator row, so the group minimum and
//                         maximum are thread-local.
//
// Warp roles: one TMA producer thread, one MMA issuer thread, epilogue warps that read the accumulator with
// tcgen05.ld and, in the first kernel, two converter warps that turn the INT4 codes of the projection matrix
// into the bf16 operand tile inside shared memory (Sec. 3.3: the projection is stored in INT4 and dequantized
// where it is used).  The accumulator is double buffered in tensor memory, so the epilogue of a tile overlaps
// the main loop of the next one.  Everything global the epilogue touches goes through shared memory in the
// 128-byte TMA swizzle: a thread reads/writes its own row with 16-byte accesses without bank
// conflicts, and global traffic stays fully coalesced.
//
// Every barrier wait is bounded; on expiry the kernel raises QG_DEV_WAIT_EXPIRED in the status word,
// stops taking tiles, releases its tensor memory and returns.
#include <cstdio>
#include <cstring>
#include <algorithm>
#include <queue>
#include <type_traits>
#include <vector>

#include "sm100_ptx.cuh"
#include "tensor_map.cuh"
#include "step_epilogue.cuh"

namespace qg {

namespace {

using namespace ptx;

constexpr int kBK = 64;                 // K extent of one pipeline stage (elements)
constexpr int kBoxBytes = 64 * kBK * 2; // one TMA box of an operand: 64 x kBK bf16 = 8 KB
constexpr int kTileM = 128;             // accumulator rows (TMEM lanes)
constexpr int kChunk = 32;              // accumulator columns per tcgen05.ld

// One matrix of the step, as the kernels see it.  Tensor maps (row-major tensors, inner extent first):
//   mapP    P~  bf16 [m][r]       box 64 x 64, swizzle 128   A operand of the projection (2-D, exact bounds)
//   mapG    G   bf16 [m][ldg]     box 64 x 64, swizzle 128   B operand of the projection (2-D, exact bounds)
//   mapP3   P~  as (64, m, r/64)  box 64 x 64 x 2            the same operand tiles in ONE copy each: an
//   mapG3   G   as (64, m, n/64)  box 64 x 64 x BN/64        MN-major tile is a row of 64-column chunks, and
//   mapN3   N_b as (64, r, ldn/64) box 64 x 64 x 4           the third dimension walks the chunks
//   mapPk   P~  bf16 [m][r]       box 64 x 128, swizzle 128  A operand of the back-projection (K-major)
// The 3-D views hold whole chunks only; a tile that touches a ragged last chunk (r or n not a multiple
// of 64) is loaded chunk by chunk through the 2-D maps, whose bounds are exact.  One copy per operand
// matters because a single thread issues them: with six copies per K block that thread, not the tensor
// pipe, set the pace.
//   mapW    int8 [m][ldw]         box 128 x 128, swizzle 128 load of the requantizing epilogue
//   mapM, mapV  fp32 [r][ldmv]    box 32 x 16, swizzle 128   the Adam epilogue's reads of the old moments
// Everything the epilogues write (M, V, N_b, the INT8 codes, scales and zero points) goes out with plain
// vector stores: a TMA store clips at 16-byte granularity and would spill into the row padding of a ragged
// matrix.
struct alignas(64) TcProblem {
  CUtensorMap mapP, mapG, mapP3, mapG3, mapG3h, mapN3, mapN3h, mapPk, mapW, mapM, mapV;
  CUtensorMap mapGk, mapQk;            // right projection: G and Q~ as K-major B operands (see below)
  float* w_scales;
  float* w_zeros;
  float* dbgR;
  float* dbgN;
  float* dbgW;
  uint16_t* dbgNb;                     // test tap: N_b with the pitch of the moments
  float* M;
  float* V;
  int8_t* w_codes;
  uint16_t* nb;                        // N_b, bf16 r x ldn (scratch)
  int64_t ldmv, ldw, ldn;
  int32_t m, n, r, ngroups;
  // The projection kernel sees a K extent and a column extent: (m, n) for R = P~^T G, and (n, m) for the
  // right-hand form R^T = Q~^T G^T, where the same kernel runs on the transposed gradient: G itself (m x n,
  // row-major) is then the B operand with K contiguous (mapGk, box 64 x 128 rows), the moments and N_b are
  // r x m, and the back-projection D = N_b^T Q~^T takes N_b as an MN-major A (mapN3h) and Q~ (n x r) as a
  // K-major B (mapQk, box 64 x 256 rows).
  int32_t right, k1_k, k1_n;
  // 8-bit moments: M, V point to int8 / uint8 codes (pitch ldmv bytes), mapM / mapV are byte maps (box 32 x 16,
  // no swizzle), m_scale / v_scale hold one fp32 scale per block of 32 columns of a row ([r][nsb]).
  int32_t state8, nsb;
  float* m_scale;
  float* v_scale;
  // The projection's A operand converted in the kernel: the INT4 codes, scales and zero points of the projection
  // matrix (row pitch in bytes, groups per row) and where the bf16 copy for the back-projection goes.  fuse_a = 0
  // (2- or 8-bit codes, a rank that is not a multiple of 128): the tile comes by TMA from a bf16 copy made beforehand.
  const uint8_t* p_codes;
  const float* p_scales;
  const float* p_zeros;
  uint16_t* pt;
  int64_t p_row_bytes;
  int32_t p_ngroups, fuse_a;
  int32_t r_whole, n_whole;            // r, n rounded down to whole 64-column chunks (extent of the 3-D views)
  uint32_t seed_lo, seed_hi;           // stochastic-rounding key of this matrix
  int32_t k1_rblocks, k1_tiles;
  int32_t k1_rpairs, k1p_tiles;        // the same in 256-row blocks of r (256-column tiles), for CTA pairs
  int32_t k2_mblocks, k2_tiles;
  int32_t k2_mpairs, k2p_tiles;        // the same in 256-row blocks, for CTA pairs
};
static_assert(sizeof(TcProblem) <= 2048, "TcProblem must fit the kernel parameter space");

// The tiles one CTA works through.  A single matrix is walked round-robin (tile = block, block + grid, ...);
// a plan carries a precomputed list per CTA, (problem, tile within the problem) pairs in entries
// [start[block], start[block + 1]): tiles differ in cost by the K extent of their matrix, and a
// longest-first assignment on the host keeps the CTAs level where round-robin left the slowest one with
// 1.6 times the average work.
struct TileSchedule {
  const int32_t* start;
  const int2* items;
  int32_t ctas;          // CTAs that share one list (2 when the kernel runs as CTA pairs)
};

template <bool SINGLE>
struct TileWalk {
  int idx, end, stride;
  const int2* items;
  __device__ TileWalk(const TileSchedule& s, int total_tiles) {
    if (SINGLE) { idx = blockIdx.x; end = total_tiles; stride = gridDim.x; items = nullptr; }
    else { idx = s.start[blockIdx.x / s.ctas]; end = s.start[blockIdx.x / s.ctas + 1]; stride = 1; items = s.items; }
  }
  __device__ bool valid() const { return idx < end; }
  __device__ bool has_next() const { return idx + stride < end; }
  __device__ int2 at(int i) const { return SINGLE ? make_int2(0, i) : items[i]; }
  __device__ int2 cur() const { return at(idx); }
  __device__ int2 next() const { return at(idx + stride); }
  __device__ void advance() { idx += stride; }
};

__device__ __forceinline__ void raise_wait_expired(int32_t* status) {
  if (status) atomicOr(status, QG_DEV_WAIT_EXPIRED);
}

constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23: adding it leaves an integer in the low mantissa bits

__device__ __forceinline__ float min3(float a, float b, float c) {
  float d;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ============================================================================================
// Kernel 1: projection + Adam
// ============================================================================================
// MVS: slots of the M/V rings (0: three while a stage is at most 32 KB, else two).  Fewer slots leave room for one
// more operand stage, which pays when the main loop is long (LLaMA-7B: K = 4096 .. 11008) and costs a little when it
// is short.
template <int BN, int CTAS = 1, int MVS = 0>
struct K1Smem {
  static constexpr int kABytes = 2 * kBoxBytes;            // 128 (r) x 64 (m) bf16
  static constexpr int kBBytes = (BN / 64 / CTAS) * kBoxBytes;   // this CTA's share of BN (n) x 64 (m) bf16
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kEpiWarps = 8;                      // 4 lane quarters x 2 halves of 16 lanes
  // every epilogue warp stages its own 16 rows x 32 columns of M and of V per accumulator chunk, kMvSlots
  // chunks deep, through TMA
  static constexpr int kMvSlots = MVS > 0 ? MVS : (kStageBytes > 32 * 1024 ? 2 : 3);
  static constexpr int kMvArrayBytes = 16 * kChunk * 4;    // 2 KB: one array's piece of a chunk
  static constexpr int kMvSlotBytes = 2 * kMvArrayBytes;   // M then V
  static constexpr int kMvBytes = kEpiWarps * kMvSlots * kMvSlotBytes;
  static constexpr int kStages = (224 * 1024 - kMvBytes) / kStageBytes;
  static constexpr int kMvOffset = kStages * kStageBytes;
  static constexpr int kBarOffset = kMvOffset + kMvBytes;
  static constexpr int kBytes = kBarOffset + 512 + 1024;   // barriers + slack for 1024-byte alignment
  static constexpr int kConvWarps = 2;                      // one thread per K row of a stage converts 128 codes
  static constexpr int kThreads = 64 + kEpiWarps * 32 + kConvWarps * 32;
};

// The Adam update of Sec. 3.5: M <- b1 M + (1-b1) R, V <- b2 V + (1-b2) R^2,
// N = (M / (1 - b1^t)) / (sqrt(V / (1 - b2^t)) + eps)   (Kingma & Ba; eps outside the root).
// Constants of the Adam update in the form the epilogue uses them: with k_v = bias1^2 / bias2 and
// eps_b = eps * bias1,  N = (M / bias1) / (sqrt(V / bias2) + eps) = M / (sqrt(V * k_v) + eps_b).
struct AdamConsts {
  float2 b1, b2, omb1, omb2, kv, epsb;
};

// Adam on two adjacent elements: m, v are updated in place, the direction is returned.
__device__ __forceinline__ float2 adam2(const AdamConsts& c, float2 r, float2& m, float2& v) {
  m = fma2(c.b1, m, mul2(c.omb1, r));
  v = fma2(c.b2, v, mul2(mul2(c.omb2, r), r));
  const float2 q = mul2(v, c.kv);
  const float2 den = add2(make_float2(sqrt_approx(q.x), sqrt_approx(q.y)), c.epsb);
  return make_float2(__fdividef(m.x, den.x), __fdividef(m.y, den.y));
}

// One K row of the projection's A tile: 128 INT4 codes (64 bytes, `c`) of row `ct` of a stage -> bf16((q - z) * s)
// in the 128-byte-swizzled MN-major layout (`sA` = the row's base in the stage: two 64-column slabs of 8 KB, the
// 16-byte piece p of a row stored at p ^ (row % 8)), and, if `gout` is given, to the same row of the bf16 copy in
// global memory.  FAST: the stored nibble (code + 8) is dropped into the mantissa of 2^23 and (2^23 + 8 + z)
// subtracted: q - z exactly, without an integer-to-float conversion, for |z| < 2^22.
template <bool FAST>
__device__ __forceinline__ void convert_p_row(const uint4 (&c)[4], float s_cur, float z_cur, uint8_t* sA, int ct, uint16_t* gout) {
  const float cz = 8388616.0f + z_cur;
  const float2 mcz = make_float2(-cz, -cz), s2 = make_float2(s_cur, s_cur);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t w4[4] = {c[j].x, c[j].y, c[j].z, c[j].w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t lo4 = w4[i] & 0x0F0F0F0Fu, hi4 = (w4[i] >> 4) & 0x0F0F0F0Fu;   // even and odd columns, one per byte
      uint32_t o[4];
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        float2 v;
        if (FAST) {
          v = mul2(add2(make_float2(__uint_as_float(__byte_perm(lo4, 0x4B000000u, 0x7650 + b)),
                                    __uint_as_float(__byte_perm(hi4, 0x4B000000u, 0x7650 + b))), mcz), s2);
        } else {
          v.x = __fmul_rn(__fsub_rn((float)((int)((lo4 >> (8 * b)) & 0xFu) - 8), z_cur), s_cur);
          v.y = __fmul_rn(__fsub_rn((float)((int)((hi4 >> (8 * b)) & 0xFu) - 8), z_cur), s_cur);
        }
        const __nv_bfloat162 h2 = __floats2bfloat162_rn(v.x, v.y);
        o[b] = *reinterpret_cast<const uint32_t*>(&h2);
      }
      const uint4 out = make_uint4(o[0], o[1], o[2], o[3]);
      // columns 32 j + 8 i .. + 7 of the rank block: slab j / 2, piece (j % 2) * 4 + i of the row
      *reinterpret_cast<uint4*>(sA + (j >> 1) * kBoxBytes + (((((j & 1) << 2) + i) ^ (ct & 7)) << 4)) = out;
      if (gout) *reinterpret_cast<uint4*>(gout + 32 * j + 8 * i) = out;
    }
  }
}

// The epilogue reads the accumulator in the 16-lane x 256-bit shape: thread t holds, per group of
// eight columns, the column pair 2(t%4), 2(t%4)+1 of rows t/4 and t/4 + 8.  A quad of threads therefore
// covers 32 contiguous bytes of a row of M, V (fp32): every global store of the epilogue writes whole
// 32-byte sectors straight from registers.  The old M, V come the other way through shared memory, by
// TMA, several chunks ahead (see the epilogue).
// S8: the instance that also knows the 8-bit storage of the moments (it costs registers, so launches whose
// matrices all keep fp32 moments take the instance without it).
template <int BN, bool SINGLE, int CTAS, bool S8 = false, int MVS = 0>
__global__ void __launch_bounds__(K1Smem<BN>::kThreads, 1)
project_adam_kernel(const __grid_constant__ TcProblem single, const TcProblem* __restrict__ table,
                    const TileSchedule sched, int total_tiles, const StepScalars sc, int32_t* __restrict__ status,
                    const int conv_active) {
  static_assert(CTAS == 1 || (!SINGLE && BN == 256), "CTA pairs run from a plan, on 256-column tiles");
  using S = K1Smem<BN, CTAS, MVS>;
  const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0u;   // 0 = the pair's leader, which issues the MMAs
  constexpr int BNC = BN / CTAS;                 // columns of the B tile this CTA stages
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stage_base = smem;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::kBarOffset);
  uint64_t* full = bars;                         // [kStages]
  uint64_t* empty = bars + S::kStages;           // [kStages]
  uint64_t* acc_full = bars + 2 * S::kStages;    // [2]
  uint64_t* acc_empty = acc_full + 2;            // [2]
  uint64_t* mv_full = acc_empty + 2;             // [kEpiWarps][kMvSlots]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(mv_full + S::kEpiWarps * S::kMvSlots);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const TcProblem* probs = SINGLE ? &single : table;

  if (threadIdx.x == 0) {
    // a stage is full once the producer's copies have landed and, in a launch some matrix of which has its A tile
    // converted in the kernel (conv_active), the converter warps (of both CTAs of a pair) have written, or waived,
    // their part of it
    for (int i = 0; i < S::kStages; ++i) {
      mbar_init(&full[i], 1 + (conv_active ? CTAS * S::kConvWarps : 0));
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], CTAS * S::kEpiWarps); }
    for (int i = 0; i < S::kEpiWarps * S::kMvSlots; ++i) mbar_init(&mv_full[i], 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    if (CTAS == 2) { tmem_alloc_pair(tmem_slot, 2 * BN); tmem_relinquish_pair(); }
    else { tmem_alloc(tmem_slot, 2 * BN); tmem_relinquish(); }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (CTAS == 2) cluster_sync_all();              // the peer's barriers exist before anything signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // tile -> (r block, n block) of its problem; consecutive tiles share the n block, so that the G tile
  // one of them brings from HBM serves the others from L2.  A pair takes two adjacent r blocks (this CTA the
  // one of its rank) and splits the columns of the G tile: each CTA stages its own 128 rows of P~^T and its
  // half of G, the leader's MMA (M = 256) reads both halves.

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (TileWalk<SINGLE> tw(sched, total_tiles); ok && tw.valid(); tw.advance()) {
        const int2 item = tw.cur();
        const TcProblem* p = probs + item.x;
        const int local = item.y, rblocks = CTAS == 2 ? p->k1_rpairs : p->k1_rblocks;
        const int r0 = (local % rblocks) * (CTAS * kTileM) + (int)rank * kTileM;
        const int n0 = (local / rblocks) * BN + (int)rank * BNC;      // first column this CTA stages
        const int kblocks = (p->k1_k + kBK - 1) / kBK;
        const bool right = p->right != 0;
        const CUtensorMap* mapP = &p->mapP;
        const CUtensorMap* mapG = &p->mapG;
        const CUtensorMap* mapP3 = &p->mapP3;
        const CUtensorMap* mapG3 = CTAS == 2 ? &p->mapG3h : &p->mapG3;
        // whole-chunk tiles take one 3-D copy per operand; chunks past the end of a 3-D view read as zero
        const bool a3 = (p->r_whole == p->r) || (r0 + kTileM <= p->r_whole);
        const bool b3 = (p->n_whole == p->k1_n) || (n0 + BNC <= p->n_whole);
        const bool fuse_a = p->fuse_a != 0;            // the converter warps write the A tile: nothing to copy
        const uint32_t tx_bytes = fuse_a ? S::kBBytes : S::kStageBytes;
        // (An L2 prefetch of G a few K blocks ahead was tried and removed: the extra TMA instruction per K
        // block cost the single producer thread more than the hidden latency was worth.)
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          const uint32_t ph = (it / S::kStages) & 1;
          if (!mbar_wait(&empty[s], ph ^ 1)) { ok = false; break; }
          uint8_t* sA = stage_base + s * S::kStageBytes;
          uint8_t* sB = sA + S::kABytes;
          if (CTAS == 2) {
            // the leader's barrier counts the bytes of both CTAs; every copy lands in the issuing CTA only
            if (rank == 0) mbar_arrive_expect_tx(&full[s], 2 * tx_bytes);
            const uint32_t lead_full = mapa_u32(smem_u32(&full[s]), 0);
            if (fuse_a) {
            } else if (a3) {
              tma_load_3d_pair(sA, mapP3, lead_full, 0, kb * kBK, r0 / 64);
            } else {
#pragma unroll
              for (int h = 0; h < 2; ++h) tma_load_2d_pair(sA + h * kBoxBytes, mapP, lead_full, r0 + 64 * h, kb * kBK);
            }
            if (right) {                               // G rows n0.. as a K-major tile of 128 rows
              tma_load_2d_pair(sB, &p->mapGk, lead_full, kb * kBK, n0);
            } else if (b3) {
              tma_load_3d_pair(sB, mapG3, lead_full, 0, kb * kBK, n0 / 64);
            } else {
#pragma unroll
              for (int h = 0; h < BNC / 64; ++h) tma_load_2d_pair(sB + h * kBoxBytes, mapG, lead_full, n0 + 64 * h, kb * kBK);
            }
          } else {
            mbar_arrive_expect_tx(&full[s], tx_bytes);
            if (fuse_a) {
            } else if (a3) {
              tma_load_3d(sA, mapP3, &full[s], 0, kb * kBK, r0 / 64);
            } else {
#pragma unroll
              for (int h = 0; h < 2; ++h) tma_load_2d(sA + h * kBoxBytes, mapP, &full[s], r0 + 64 * h, kb * kBK);
            }
            if (right) {
#pragma unroll
              for (int h = 0; h < BN / 128; ++h) tma_load_2d(sB + h * 2 * kBoxBytes, &p->mapGk, &full[s], kb * kBK, n0 + 128 * h);
            } else if (b3) {
              tma_load_3d(sB, mapG3, &full[s], 0, kb * kBK, n0 / 64);
            } else {
#pragma unroll
              for (int h = 0; h < BN / 64; ++h) tma_load_2d(sB + h * kBoxBytes, mapG, &full[s], n0 + 64 * h, kb * kBK);
            }
          }
        }
      }
      if (!ok) raise_wait_expired(status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc_left = umma_idesc_bf16(CTAS * kTileM, BN, true, true);
      constexpr uint32_t idesc_right = umma_idesc_bf16(CTAS * kTileM, BN, true, false);   // B with K contiguous
      const uint64_t desc_a0 = umma_smem_desc_sw128(smem_u32(stage_base), kBoxBytes, 1024);
      const uint64_t desc_b0 = umma_smem_desc_sw128(smem_u32(stage_base) + S::kABytes, kBoxBytes, 1024);
      const uint64_t desc_bk0 = umma_smem_desc_sw128(smem_u32(stage_base) + S::kABytes, 16, 1024);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (TileWalk<SINGLE> tw(sched, total_tiles); ok && tw.valid(); tw.advance(), ++tcount) {
        const TcProblem* p = probs + tw.cur().x;
        const int kblocks = (p->k1_k + kBK - 1) / kBK;
        const bool right = p->right != 0;
        const uint32_t idesc = right ? idesc_right : idesc_left;
        const uint64_t bstep = right ? (32 >> 4) : (2048 >> 4);   // 16 K indices further along B
        const uint32_t ab = tcount & 1;
        if (!(CTAS == 2 ? mbar_wait_cluster(&acc_empty[ab], ((tcount >> 1) & 1) ^ 1)
                        : mbar_wait(&acc_empty[ab], ((tcount >> 1) & 1) ^ 1))) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + ab * BN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          if (!(CTAS == 2 ? mbar_wait_cluster(&full[s], (it / S::kStages) & 1) : mbar_wait(&full[s], (it / S::kStages) & 1))) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          // both operands are MN-major: 16 K indices = two 8-index groups of 1024 bytes each; the start
          // address field counts 16-byte units, so a stage or K step is an add on the descriptor
          const uint64_t da = desc_a0 + (uint64_t)((s * S::kStageBytes) >> 4);
          const uint64_t db = (right ? desc_bk0 : desc_b0) + (uint64_t)((s * S::kStageBytes) >> 4);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            if (CTAS == 2) umma_bf16_pair(d_tmem, da + k * (2048 >> 4), db + k * bstep, idesc, (kb | k) != 0);
            else umma_bf16(d_tmem, da + k * (2048 >> 4), db + k * bstep, idesc, (kb | k) != 0);
          }
          if (CTAS == 2) umma_commit_pair(&empty[s]); else umma_commit(&empty[s]);
        }
        if (ok) { if (CTAS == 2) umma_commit_pair(&acc_full[ab]); else umma_commit(&acc_full[ab]); }
      }
      if (!ok) raise_wait_expired(status);
    }
  } else if (warp >= 2 + S::kEpiWarps) {
    // ------------------------------------------------------------------ converters: INT4 codes -> bf16 A tile
    // P~ = bf16((q - z) * s) (App. A, the dequantization line) is formed here, K block by K block, straight in
    // the 128-byte-swizzled MN-major operand layout: thread ct owns K row ct of the stage, i.e. row kb * 64 + ct
    // of the projection matrix, and converts the 128 codes (64 bytes) of the tile's rank block: the stored nibble
    // (code + 8) is dropped into the mantissa of 2^23 and (2^23 + 8 + z) subtracted, which gives q - z exactly
    // without an integer-to-float conversion.  Codes, scale and zero point of the NEXT K block are fetched (from
    // L2: the codes of a matrix are 1/4 the size of its bf16 form) before this one is converted.  The tiles of the
    // first column block also write the converted rows to global memory, where the back-projection reads its
    // K-major operand from.
    // Off by default (conv_active = 0: these warps leave at once).  Measured on B200, LLaMA-1B shapes, one CTA per
    // tile: 1.8 us per K block with the conversion against 0.8 us without.  The kernel is bound by how many bytes
    // it keeps in flight, a stage now also waits for this warp's chain (wake-up, a load issued one K block
    // earlier that takes about 1.5 us to return under the kernel's own traffic, 450 instructions, fence, arrive),
    // and the global stores of the writer tiles delay their barrier arrivals; as CTA pairs the arrival on the
    // leader's barrier is a cluster-scope release, about 1 us each.  The separate conversion launch costs 0.2 us
    // per K block equivalent, so it stays the default until these warps take their codes through the copy
    // engine several stages ahead.
    const int ct = (int)threadIdx.x - (64 + S::kEpiWarps * 32);
    struct Pos {
      TileWalk<SINGLE> tw;
      const TcProblem* p;
      int kb, kblocks, r0;
      bool writer;
      __device__ Pos(const TileSchedule& sch, int total) : tw(sch, total), p(nullptr), kb(0), kblocks(0), r0(0), writer(false) {}
    };
    auto enter = [&](Pos& ps) {
      if (!ps.tw.valid()) return;
      const int2 item = ps.tw.cur();
      ps.p = probs + item.x;
      const int rblocks = CTAS == 2 ? ps.p->k1_rpairs : ps.p->k1_rblocks;
      ps.r0 = (item.y % rblocks) * (CTAS * kTileM) + (int)rank * kTileM;
      ps.writer = (item.y / rblocks) == 0;
      ps.kblocks = (ps.p->k1_k + kBK - 1) / kBK;
      ps.kb = 0;
    };
    auto fetch = [&](const Pos& ps, uint4 c[4], float& sc_, float& zp) {
      c[0] = c[1] = c[2] = c[3] = make_uint4(0u, 0u, 0u, 0u);
      sc_ = 0.f; zp = 0.f;                            // rows past the matrix convert to zero
      if (!ps.tw.valid() || !ps.p->fuse_a) return;
      const int64_t row = (int64_t)ps.kb * kBK + ct;
      if (row >= ps.p->k1_k) return;
      const uint4* src = reinterpret_cast<const uint4*>(ps.p->p_codes + row * ps.p->p_row_bytes + (ps.r0 >> 1));
#pragma unroll
      for (int j = 0; j < 4; ++j) c[j] = __ldg(src + j);
      const int64_t g = row * ps.p->p_ngroups + (ps.r0 >> 8);
      sc_ = __ldg(ps.p->p_scales + g);
      zp = __ldg(ps.p->p_zeros + g);
    };
    Pos pos(sched, total_tiles);
    enter(pos);
    uint4 cn[4];
    float sn, zn;
    fetch(pos, cn, sn, zn);
    uint32_t it = 0;
    bool ok = true;
    while (conv_active && ok && pos.tw.valid()) {
      const uint4 c[4] = {cn[0], cn[1], cn[2], cn[3]};
      const float s_cur = sn, z_cur = zn;
      const TcProblem* p = pos.p;
      const int kb = pos.kb, r0 = pos.r0;
      const bool writer = pos.writer;
      if (++pos.kb >= pos.kblocks) { pos.tw.advance(); enter(pos); }
      fetch(pos, cn, sn, zn);
      const int s = it % S::kStages;
      // the MMAs that read this stage are done; one lane polls, so that the warp does not crowd the barrier unit the
      // copies and commits of the pipeline go through
      if (lane == 0) ok = mbar_wait(&empty[s], ((it / S::kStages) & 1) ^ 1);
      ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
      if (!ok) break;
      if (p->fuse_a) {
        uint8_t* sA = stage_base + s * S::kStageBytes + ct * 128;
        const int64_t row = (int64_t)kb * kBK + ct;
        uint16_t* gout = (writer && row < p->k1_k) ? p->pt + row * p->r + r0 : nullptr;
        // the exact-by-construction fast form needs |z| < 2^22; a warp with a row outside that takes the plain form
        if (__all_sync(0xFFFFFFFFu, fabsf(z_cur) < 4.0e6f)) convert_p_row<true>(c, s_cur, z_cur, sA, ct, gout);
        else convert_p_row<false>(c, s_cur, z_cur, sA, ct, gout);
        fence_proxy_async_smem();                        // the MMA reads these stores through the async proxy
      }
      __syncwarp();
      if (lane == 0) {
        if (CTAS == 2) mbar_arrive_cluster(mapa_u32(smem_u32(&full[s]), 0));
        else mbar_arrive(&full[s]);
      }
      ++it;
    }
    if (!ok && lane == 0) raise_wait_expired(status);
  } else {
    // ------------------------------------------------------------------ epilogue: Adam on the tile
    const int q = warp & 3, hh = (warp - 2) >> 2;   // TMEM lane quarter of this warp, 16-lane half within it
    const int wrow = q * 32 + hh * 16;               // first of the warp's 16 tile rows
    const int lrow = wrow + (lane >> 2);             // first of the thread's two tile rows (the other: + 8)
    const int lcol = 2 * (lane & 3);                 // first column of the thread's pair within a group of 8
    const uint32_t lane_addr = (uint32_t)wrow << 16;
    AdamConsts ac;
    ac.b1 = make_float2(sc.beta1, sc.beta1); ac.b2 = make_float2(sc.beta2, sc.beta2);
    ac.omb1 = make_float2(sc.one_minus_beta1, sc.one_minus_beta1); ac.omb2 = make_float2(sc.one_minus_beta2, sc.one_minus_beta2);
    ac.kv = make_float2(sc.bias1 * sc.bias1 / sc.bias2, sc.bias1 * sc.bias1 / sc.bias2);
    ac.epsb = make_float2(sc.eps * sc.bias1, sc.eps * sc.bias1);

    // M and V reach the warp through shared memory: one TMA copy per array brings the warp's 16 rows x 32
    // columns of a chunk (rows of 128 bytes, 128-byte swizzle; columns and rows past the matrix read as
    // zero), kMvSlots chunks ahead of the one being computed and across tile boundaries.  Loads that wait
    // in registers cannot run that far ahead: a warp has six scoreboards to track them with, and a wait for
    // one chunk's registers also waits for the younger loads that share its scoreboard.
    const int ew = warp - 2;
    uint8_t* mv_base = smem + S::kMvOffset + ew * (S::kMvSlots * S::kMvSlotBytes);
    uint64_t* my_full = mv_full + ew * S::kMvSlots;
    // byte offset of the thread's column pair of 8-column group k in a staged row: 16-byte unit
    // (2k + (lane & 3) / 2) ^ (row % 8), then 8 bytes for the odd pair; both of the thread's rows have the
    // same row % 8
    const uint32_t swz = (uint32_t)(lane >> 2), half8 = (uint32_t)(lane & 1) * 8u, unit0 = (uint32_t)((lane >> 1) & 1);
    const uint32_t row_off = (uint32_t)(lane >> 2) * 128u;

    // With 8-bit moments a warp takes all 32 rows of its lane quarter and every second chunk (a thread then holds
    // one whole 32-element block of a row); with fp32 moments 16 rows and every chunk.
    struct Cursor {                                  // a (tile, chunk) position in this CTA's work list
      TileWalk<SINGLE> tw;
      const TcProblem* p;
      int c, cstep, nch, x0, y0;
      __device__ Cursor(const TileSchedule& sch, int total) : tw(sch, total), p(nullptr), c(0), cstep(1), nch(0), x0(0), y0(0) {}
    };
    auto enter_tile = [&](Cursor& cu) {
      while (cu.tw.valid()) {
        const int2 item = cu.tw.cur();
        cu.p = probs + item.x;
        const bool t8 = S8 && cu.p->state8 != 0;
        const int rblocks = CTAS == 2 ? cu.p->k1_rpairs : cu.p->k1_rblocks;
        cu.y0 = (item.y % rblocks) * (CTAS * kTileM) + (int)rank * kTileM + (t8 ? q * 32 : wrow);
        cu.x0 = (item.y / rblocks) * BN;
        cu.nch = min(BN / kChunk, (cu.p->k1_n - cu.x0 + kChunk - 1) / kChunk);
        cu.c = t8 ? hh : 0;
        cu.cstep = t8 ? 2 : 1;
        if (cu.c < cu.nch) return;
        cu.tw.advance();                             // a one-chunk tile has nothing for the warp of the odd chunks
      }
    };
    auto next_chunk = [&](Cursor& cu) {
      cu.c += cu.cstep;
      if (cu.c >= cu.nch) { cu.tw.advance(); enter_tile(cu); }
    };
    Cursor ld(sched, total_tiles);                   // the next chunk to request
    enter_tile(ld);
    uint32_t ld_slot = 0, in_flight = 0;
    auto request = [&]() {                           // one lane: the two copies of chunk `ld` into slot ld_slot
      if (lane == 0) {
        uint8_t* dst = mv_base + ld_slot * S::kMvSlotBytes;
        mbar_arrive_expect_tx(&my_full[ld_slot], (S8 && ld.p->state8) ? 2 * 32 * kChunk : S::kMvSlotBytes);
        tma_load_2d(dst, &ld.p->mapM, &my_full[ld_slot], ld.x0 + kChunk * ld.c, ld.y0);
        tma_load_2d(dst + S::kMvArrayBytes, &ld.p->mapV, &my_full[ld_slot], ld.x0 + kChunk * ld.c, ld.y0);
      }
      ld_slot = (ld_slot + 1 == (uint32_t)S::kMvSlots) ? 0u : ld_slot + 1;
      ++in_flight;
      next_chunk(ld);
    };
#pragma unroll 1
    for (int i = 0; i < S::kMvSlots && ld.tw.valid(); ++i) request();

    uint32_t tcount = 0, slot = 0, slot_phase = 0;
    bool ok = true;
    for (TileWalk<SINGLE> tw(sched, total_tiles); ok && tw.valid(); tw.advance(), ++tcount) {
      const int2 item = tw.cur();
      const TcProblem* p = probs + item.x;
      const int local = item.y, rblocks = CTAS == 2 ? p->k1_rpairs : p->k1_rblocks;
      const int r0 = (local % rblocks) * (CTAS * kTileM) + (int)rank * kTileM, n0 = (local / rblocks) * BN;
      const int pn = p->k1_n;
      const int nch = min(BN / kChunk, (pn - n0 + kChunk - 1) / kChunk);
      const int cmax = pn - n0 - lcol;               // offset `off` (from n0 + lcol) is a valid column iff off < cmax
      const int64_t ldmv = p->ldmv, ldn = p->ldn;
      float* Mr[2]; float* Vr[2]; uint16_t* Nr[2]; float* tapR[2]; float* tapN[2]; uint16_t* tapNb[2];
      bool rok[2];
#pragma unroll
      for (int a = 0; a < 2; ++a) {
        const int64_t gr = r0 + lrow + 8 * a;
        rok[a] = gr < p->r;
        Mr[a] = p->M + gr * ldmv + n0 + lcol;
        Vr[a] = p->V + gr * ldmv + n0 + lcol;
        Nr[a] = p->nb + gr * ldn + n0 + lcol;
        tapR[a] = p->dbgR ? p->dbgR + gr * ldmv + n0 + lcol : nullptr;
        tapN[a] = p->dbgN ? p->dbgN + gr * ldmv + n0 + lcol : nullptr;
        tapNb[a] = p->dbgNb ? p->dbgNb + gr * ldmv + n0 + lcol : nullptr;
      }
      // interior tiles (every row and column valid, no test taps) take a path without per-access predicates
      const bool s8 = S8 && p->state8 != 0;
      const bool whole = (r0 + kTileM <= p->r) && (n0 + BN <= pn) && p->dbgR == nullptr && p->dbgN == nullptr && p->dbgNb == nullptr;
      const bool interior = whole;
      const uint32_t ab = tcount & 1;
      if (s8) {
        // ---- 8-bit moments: thread = one row of the lane quarter, chunk = one 32-element block of that row
        const int64_t gr = r0 + q * 32 + lane;
        const bool rok8 = gr < p->r;
        int8_t* M8 = reinterpret_cast<int8_t*>(p->M) + gr * ldmv + n0;
        uint8_t* V8 = reinterpret_cast<uint8_t*>(p->V) + gr * ldmv + n0;
        float* msc = p->m_scale + gr * p->nsb;
        float* vsc = p->v_scale + gr * p->nsb;
        uint16_t* Nrow = p->nb + gr * ldn + n0;
        float* tR = p->dbgR ? p->dbgR + gr * ldmv + n0 : nullptr;
        float* tN = p->dbgN ? p->dbgN + gr * ldmv + n0 : nullptr;
        uint16_t* tNb = p->dbgNb ? p->dbgNb + gr * ldmv + n0 : nullptr;
        const int cvalid = pn - n0;                  // columns of the tile inside the matrix
        float ms_next = 0.f, vs_next = 0.f;          // the block scales, fetched one chunk ahead
        auto fetch_scales = [&](int c) {
          const int blk = (n0 + kChunk * c) >> 5;
          ms_next = rok8 ? __ldg(msc + blk) : 0.f;
          vs_next = rok8 ? __ldg(vsc + blk) : 0.f;
        };
        if (hh < nch) fetch_scales(hh);
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(&acc_full[ab], (tcount >> 1) & 1));
        if (!ok) break;
        tc_fence_after_sync();
        auto release_acc = [&]() {                   // every read of this accumulator buffer has landed
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            if (CTAS == 2) mbar_arrive_cluster(mapa_u32(smem_u32(&acc_empty[ab]), 0));
            else mbar_arrive(&acc_empty[ab]);
          }
        };
        if (hh >= nch) release_acc();
#pragma unroll 1
        for (int c = hh; c < nch; c += 2) {
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(&my_full[slot], slot_phase));
          if (!ok) break;
          --in_flight;
          // the 32 + 32 codes of the thread's block (rows of 32 bytes, no swizzle)
          const uint4* src8 = reinterpret_cast<const uint4*>(mv_base + slot * S::kMvSlotBytes + lane * kChunk);
          const uint4 mc4[2] = {src8[0], src8[1]};
          const uint4 vc4[2] = {src8[S::kMvArrayBytes / 16], src8[S::kMvArrayBytes / 16 + 1]};
          const float ms = ms_next, vs = vs_next;
          if (c + 2 < nch) fetch_scales(c + 2);
          if (++slot == (uint32_t)S::kMvSlots) { slot = 0; slot_phase ^= 1u; }
          fence_proxy_async_smem();
          __syncwarp();
          if (ld.tw.valid()) request();

          uint32_t acc[32];
          tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + ab * BN + c * kChunk, acc);
          tmem_ld_wait();
          if (c + 2 >= nch) release_acc();

          const uint32_t mw[8] = {mc4[0].x, mc4[0].y, mc4[0].z, mc4[0].w, mc4[1].x, mc4[1].y, mc4[1].z, mc4[1].w};
          const uint32_t vw[8] = {vc4[0].x, vc4[0].y, vc4[0].z, vc4[0].w, vc4[1].x, vc4[1].y, vc4[1].z, vc4[1].w};
          const float stepm = __fmul_rn(ms, 1.0f / 127.0f);
          const float2 stepm2 = make_float2(stepm, stepm), vs2 = make_float2(vs, vs);
          const float2 c255 = make_float2(1.0f / 255.0f, 1.0f / 255.0f);
          const float2 bias_m = make_float2(-8388736.0f, -8388736.0f), bias_v = make_float2(-8388608.0f, -8388608.0f);
          const bool chunk_whole = rok8 && kChunk * c + kChunk <= cvalid;
          const bool taps = tR != nullptr || tN != nullptr || tNb != nullptr;
          float2 mm[16], vv[16];
          float mxm = 0.f, mxv = 0.f;
          uint32_t nbq[4];                            // the bf16 direction of eight columns, stored 16 bytes at a time
#pragma unroll
          for (int k = 0; k < 8; ++k) {               // word k: columns 4k .. 4k+3 of the block
            const uint32_t mcw = mw[k] ^ 0x80808080u;
            uint32_t* nbw = nbq + 2 * (k & 1);
#pragma unroll
            for (int b = 0; b < 2; ++b) {
              const int j = 2 * k + b;                // column pair 2j, 2j+1
              // a byte dropped into the mantissa of 2^23 is the float 2^23 + byte: no integer-to-float conversion
              const float2 mq = make_float2(__uint_as_float(__byte_perm(mcw, 0x4B000000u, 0x7650 + 2 * b)),
                                            __uint_as_float(__byte_perm(mcw, 0x4B000000u, 0x7651 + 2 * b)));
              mm[j] = mul2(add2(mq, bias_m), stepm2);                                   // code = byte - 128
              const float2 vq = make_float2(__uint_as_float(__byte_perm(vw[k], 0x4B000000u, 0x7650 + 2 * b)),
                                            __uint_as_float(__byte_perm(vw[k], 0x4B000000u, 0x7651 + 2 * b)));
              const float2 w = mul2(add2(vq, bias_v), c255);
              vv[j] = mul2(mul2(w, w), vs2);
              const float2 rr = make_float2(__uint_as_float(acc[2 * j]), __uint_as_float(acc[2 * j + 1]));
              const float2 nn = adam2(ac, rr, mm[j], vv[j]);
              const __nv_bfloat162 nb2 = __floats2bfloat162_rn(nn.x, nn.y);
              nbw[b] = *reinterpret_cast<const uint32_t*>(&nb2);
              mxm = max3(mxm, fabsf(mm[j].x), fabsf(mm[j].y));
              mxv = max3(mxv, vv[j].x, vv[j].y);
              if (taps && rok8) {
                const int off = kChunk * c + 2 * j;
#pragma unroll
                for (int e = 0; e < 2; ++e)
                  if (off + e < cvalid) {
                    if (tR) tR[off + e] = e ? rr.y : rr.x;
                    if (tN) tN[off + e] = e ? nn.y : nn.x;
                    if (tNb) tNb[off + e] = (uint16_t)(nbw[b] >> (16 * e));
                  }
              }
            }
            if (chunk_whole) {
              if (k & 1) *reinterpret_cast<uint4*>(Nrow + kChunk * c + 4 * (k - 1)) = make_uint4(nbq[0], nbq[1], nbq[2], nbq[3]);
            } else if (rok8) {
#pragma unroll
              for (int e = 0; e < 4; ++e)
                if (kChunk * c + 4 * k + e < cvalid) Nrow[kChunk * c + 4 * k + e] = (uint16_t)(nbw[e >> 1] >> (16 * (e & 1)));
            }
          }
          // 8-bit storage of the new moments: scale = the block's largest |M'| resp. V'; M' linear in [-127, 127],
          // V' by the square-root law in [0, 255]; every operation a single binary32 one, as on the reference side.
          // Reciprocals and roots by the approximate units (a few ulp): a code can differ from the correctly
          // rounded one only when the scaled value sits within ~1e-5 of a rounding boundary.
          const float invm = mxm > 0.f ? __fdividef(127.0f, mxm) : 0.f;
          const float invv = mxv > 0.f ? __fdividef(1.0f, mxv) : 0.f;
          if (!rok8) continue;
          const int blk = (n0 + kChunk * c) >> 5;
          if (kChunk * c < cvalid) { msc[blk] = mxm; vsc[blk] = mxv; }
          uint32_t mo[8], vo[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            // rint(t) sits in the low mantissa bits of t + 1.5 * 2^23; |t| <= 127 (+ a few ulp) resp. 0 <= t <= 255
            // by construction of the scales, so the low byte is the code
            uint32_t mq4[4], vq4[4];
#pragma unroll
            for (int b = 0; b < 2; ++b) {
              const float2 m2 = mm[2 * k + b], v2 = vv[2 * k + b];
              mq4[2 * b] = __float_as_uint(__fadd_rn(__fmul_rn(m2.x, invm), kMagic));
              mq4[2 * b + 1] = __float_as_uint(__fadd_rn(__fmul_rn(m2.y, invm), kMagic));
              vq4[2 * b] = __float_as_uint(__fadd_rn(__fmul_rn(sqrt_approx(__fmul_rn(v2.x, invv)), 255.0f), kMagic));
              vq4[2 * b + 1] = __float_as_uint(__fadd_rn(__fmul_rn(sqrt_approx(__fmul_rn(v2.y, invv)), 255.0f), kMagic));
            }
            mo[k] = __byte_perm(__byte_perm(mq4[0], mq4[1], 0x0040), __byte_perm(mq4[2], mq4[3], 0x0040), 0x5410);
            vo[k] = __byte_perm(__byte_perm(vq4[0], vq4[1], 0x0040), __byte_perm(vq4[2], vq4[3], 0x0040), 0x5410);
          }
          if (chunk_whole) {
            uint4* md = reinterpret_cast<uint4*>(M8 + kChunk * c);
            uint4* vd = reinterpret_cast<uint4*>(V8 + kChunk * c);
            md[0] = make_uint4(mo[0], mo[1], mo[2], mo[3]); md[1] = make_uint4(mo[4], mo[5], mo[6], mo[7]);
            vd[0] = make_uint4(vo[0], vo[1], vo[2], vo[3]); vd[1] = make_uint4(vo[4], vo[5], vo[6], vo[7]);
          } else {
#pragma unroll
            for (int e = 0; e < kChunk; ++e)
              if (kChunk * c + e < cvalid) {
                M8[kChunk * c + e] = (int8_t)((mo[e >> 2] >> (8 * (e & 3))) & 0xFFu);
                V8[kChunk * c + e] = (uint8_t)((vo[e >> 2] >> (8 * (e & 3))) & 0xFFu);
              }
          }
        }
        continue;
      }

      ok = __all_sync(0xFFFFFFFFu, mbar_wait(&acc_full[ab], (tcount >> 1) & 1));
      if (!ok) break;
      tc_fence_after_sync();
#pragma unroll 1
      for (int c = 0; c < nch; ++c) {
        // this chunk's M and V from the warp's slot into registers (index 2k + a), then the slot goes back
        // to the copy engine for the chunk kMvSlots further on
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(&my_full[slot], slot_phase));
        if (!ok) break;
        --in_flight;
        float2 sm[8], sv[8];
        {
          const uint8_t* src = mv_base + slot * S::kMvSlotBytes + row_off + half8;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint32_t u = (((uint32_t)(2 * k) + unit0) ^ swz) << 4;
#pragma unroll
            for (int a = 0; a < 2; ++a) {
              sm[2 * k + a] = *reinterpret_cast<const float2*>(src + a * 1024 + u);
              sv[2 * k + a] = *reinterpret_cast<const float2*>(src + S::kMvArrayBytes + a * 1024 + u);
            }
          }
        }
        if (++slot == (uint32_t)S::kMvSlots) { slot = 0; slot_phase ^= 1u; }
        fence_proxy_async_smem();
        __syncwarp();
        if (ld.tw.valid()) request();

        uint32_t acc[16];
        tmem_ld_16x256b_x4(tmem_base + lane_addr + ab * BN + c * kChunk, acc);
        tmem_ld_wait();
        if (c + 1 == nch) {                           // every read of this accumulator buffer has landed
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            if (CTAS == 2) mbar_arrive_cluster(mapa_u32(smem_u32(&acc_empty[ab]), 0));
            else mbar_arrive(&acc_empty[ab]);
          }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
          for (int a = 0; a < 2; ++a) {
            const int off = kChunk * c + 8 * k;
            float2 mm = sm[2 * k + a], vv = sv[2 * k + a];
            const float2 rr = make_float2(__uint_as_float(acc[4 * k + 2 * a]), __uint_as_float(acc[4 * k + 2 * a + 1]));
            const float2 nn = adam2(ac, rr, mm, vv);
            const __nv_bfloat162 nb2 = __floats2bfloat162_rn(nn.x, nn.y);
            if (interior) {
              __stcs(reinterpret_cast<float2*>(Mr[a] + off), mm);
              __stcs(reinterpret_cast<float2*>(Vr[a] + off), vv);
              *reinterpret_cast<__nv_bfloat162*>(Nr[a] + off) = nb2;
            } else if (rok[a]) {
              if (off + 1 < cmax) {
                __stcs(reinterpret_cast<float2*>(Mr[a] + off), mm);
                __stcs(reinterpret_cast<float2*>(Vr[a] + off), vv);
                *reinterpret_cast<__nv_bfloat162*>(Nr[a] + off) = nb2;
                if (tapR[a]) { tapR[a][off] = rr.x; tapR[a][off + 1] = rr.y; }
                if (tapN[a]) { tapN[a][off] = nn.x; tapN[a][off + 1] = nn.y; }
                if (tapNb[a]) { tapNb[a][off] = __bfloat16_as_ushort(nb2.x); tapNb[a][off + 1] = __bfloat16_as_ushort(nb2.y); }
              } else if (off < cmax) {             // odd n: the last column stands alone
                Mr[a][off] = mm.x;
                Vr[a][off] = vv.x;
                Nr[a][off] = float_to_bf16_bits(nn.x);
                if (tapR[a]) tapR[a][off] = rr.x;
                if (tapN[a]) tapN[a][off] = nn.x;
                if (tapNb[a]) tapNb[a][off] = __bfloat16_as_ushort(nb2.x);
              }
            }
          }
      }
    }
    if (!ok) {
      // a wait ran out: let the copies still on their way into this warp's slots land (bounded) before the
      // CTA gives its shared memory back
      for (; in_flight > 0; --in_flight) {
        mbar_wait(&my_full[slot], slot_phase);
        if (++slot == (uint32_t)S::kMvSlots) { slot = 0; slot_phase ^= 1u; }
      }
    }
    if (!ok && lane == 0) raise_wait_expired(status);
  }

  tc_fence_before_sync();
  __syncthreads();
  if (CTAS == 2) cluster_sync_all();              // neither CTA leaves while the other may still signal it
  if (warp == 1) {
    tc_fence_after_sync();
    if (CTAS == 2) tmem_dealloc_pair(tmem_base, 2 * BN); else tmem_dealloc(tmem_base, 2 * BN);
  }
}

// ============================================================================================
// Kernel 2: back-projection + dequantize-add + stochastic-rounding requantization
// ============================================================================================
struct K2Smem {
  static constexpr int kBN = 256;
  static constexpr int kStages = 3;
  static constexpr int kABytes = 2 * kBoxBytes;            // 128 (m) x 64 (r) bf16, K-major
  static constexpr int kBBytes = 4 * kBoxBytes;            // 256 (n) x 64 (r) bf16, MN-major
  static constexpr int kStageBytes = kABytes + kBBytes;    // 48 KB
  static constexpr int kCodeBufs = 2;
  static constexpr int kCodeBytes = kTileM * kBN;          // 32 KB of INT8 codes
  static constexpr int kBarOffset = kStages * kStageBytes + kCodeBufs * kCodeBytes;
  static constexpr int kPartOffset = kBarOffset + 256;     // float2 [4 slices][128 rows]: partial min/max
  static constexpr int kBytes = kPartOffset + 4 * kTileM * 8 + 1024;
  static constexpr int kEpiWarps = 16;                     // two groups of 4 lane quarters x 2 column slices of 128
  static constexpr int kEpiThreads = kEpiWarps * 32;
  static constexpr int kGroupWarps = 8;
  static constexpr int kGroupThreads = kGroupWarps * 32;
  static constexpr int kThreads = 64 + kEpiThreads;
};

// The same kernel run by CTA pairs: 256 (m) x 256 (n) per pair, each CTA stages its own 128 rows of A and its
// half (128 columns) of B.
struct K2PairSmem : K2Smem {
  static constexpr int kStages = 4;
  static constexpr int kBBytes = 2 * kBoxBytes;            // this CTA's 128 (n) x 64 (r) half of B
  static constexpr int kStageBytes = kABytes + kBBytes;    // 32 KB
  static constexpr int kBarOffset = kStages * kStageBytes + kCodeBufs * kCodeBytes;
  static constexpr int kPartOffset = kBarOffset + 256;
  static constexpr int kBytes = kPartOffset + 4 * kTileM * 8 + 1024;
};


// 16 consecutive pre-rounding weights W' = W^ - lr*alpha*D - lr*wd*W^, W^ = (q - z) * s, from 16 INT8
// codes and 16 accumulators.  FAST: q - z is formed without an integer-to-float conversion: the byte
// (q + 128) is dropped into the mantissa of 2^23 and (2^23 + 128 + z) subtracted, exact for |z| < 2^22.
template <bool FAST, bool NOWD>
__device__ __forceinline__ void weights16(const uint4 cw, const uint32_t* acc, float z, float s, float lr_alpha,
                                          float lr_wd, float* w) {
  const uint32_t w4[4] = {cw.x, cw.y, cw.z, cw.w};
  const float c0 = 8388736.0f + z;
  if (FAST && NOWD) {
    // the common case, two elements per instruction: (q - z), times s, minus lr*alpha*D
    const float2 mc0 = make_float2(-c0, -c0), s2 = make_float2(s, s), mla = make_float2(-lr_alpha, -lr_alpha);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t x = w4[k] ^ 0x80808080u;
#pragma unroll
      for (int b = 0; b < 4; b += 2) {
        const float2 v = make_float2(__uint_as_float(__byte_perm(x, 0x4B000000u, 0x7650 + b)),
                                     __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7651 + b)));
        const float2 wh = mul2(add2(v, mc0), s2);
        const float2 d = make_float2(__uint_as_float(acc[4 * k + b]), __uint_as_float(acc[4 * k + b + 1]));
        const float2 r = fma2(mla, d, wh);
        w[4 * k + b] = r.x;
        w[4 * k + b + 1] = r.y;
      }
    }
    return;
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t x = w4[k] ^ 0x80808080u;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      float qz;
      if (FAST) qz = __fsub_rn(__uint_as_float(__byte_perm(x, 0x4B000000u, 0x7650 + b)), c0);
      else qz = __fsub_rn((float)(int8_t)((w4[k] >> (8 * b)) & 0xFFu), z);
      const float wh = __fmul_rn(qz, s);
      w[4 * k + b] = fmaf(-lr_alpha, __uint_as_float(acc[4 * k + b]), NOWD ? wh : fmaf(-lr_wd, wh, wh));
    }
  }
}

// Stochastic rounding (Sec. 3.4) of 16 consecutive weights to codes of the new grid.  h holds the 16-bit
// uniforms of the 16 columns, two per word.  FAST: floor(t) + [frac(t) * 65536 > h] + z equals
// ceil(t - h / 65536) + z; it is formed as one add in round-up mode onto (2^23 * 1.5 + z), which leaves
// the code in the low byte.  The subtraction t - h / 65536 rounds by at most 2^-14 for |t| < 2^10, so a
// decision can differ from the exact one only within that distance of the rounding boundary.
// Four 32-bit integers -> four signed bytes with saturation (first argument in the lowest byte).
__device__ __forceinline__ uint32_t pack_sat_s8x4(int c0, int c1, int c2, int c3) {
  uint32_t hi, out;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(c3), "r"(c2), "r"(0));
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(out) : "r"(c1), "r"(c0), "r"(hi));
  return out;
}

// Philox4x32-10 with the ten round keys given (key schedule hoisted out of the per-block calls) and
// each 32 x 32 -> 64 bit product taken as one wide multiply.
__device__ __forceinline__ uint4 philox_rounds(uint4 c, const uint32_t* kx, const uint32_t* ky) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint64_t p0 = (uint64_t)c.x * 0xD2511F53ull, p1 = (uint64_t)c.z * 0xCD9E8D57ull;
    c = make_uint4((uint32_t)(p1 >> 32) ^ c.y ^ kx[i], (uint32_t)p1, (uint32_t)(p0 >> 32) ^ c.w ^ ky[i], (uint32_t)p0);
  }
  return c;
}

// Round to nearest (ties to even) of 16 consecutive weights to codes of the new grid: the ablation of
// Sec. 4.4.  FAST: rint(t) is read off the low mantissa bits of t + 1.5 * 2^23 (an even constant, so ties
// fall as in rint), the integer zero point is added to the bits, the pack saturates.
template <bool FAST>
__device__ __forceinline__ uint4 rtn_codes16(const float* w, const GroupParams& gp) {
  int code[16];
  if (FAST) {
    const float2 inv2 = make_float2(gp.inv, gp.inv), magic2 = make_float2(kMagic, kMagic);
    const int cz = (int)gp.z - 0x4B400000;
#pragma unroll
    for (int j = 0; j < 16; j += 2) {
      const float2 y = add2(mul2(make_float2(w[j], w[j + 1]), inv2), magic2);
      code[j] = __float_as_int(y.x) + cz;                   // may leave [-128, 127]: the pack saturates
      code[j + 1] = __float_as_int(y.y) + cz;
    }
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j) code[j] = (int)rtn_code<8>(w[j], gp);
  }
  uint32_t o[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) o[k] = pack_sat_s8x4(code[4 * k], code[4 * k + 1], code[4 * k + 2], code[4 * k + 3]);
  return make_uint4(o[0], o[1], o[2], o[3]);
}

template <bool FAST>
__device__ __forceinline__ uint4 sr_codes16(const float* w, const GroupParams& gp, const uint32_t h[8]) {
  int code[16];
  const float mz = (kMagic + 128.0f) + gp.z;
  if (FAST) {
    const float2 inv2 = make_float2(gp.inv, gp.inv), mz2 = make_float2(mz, mz);
#pragma unroll
    for (int j = 0; j < 16; j += 2) {
      // 128 + h / 65536 of the two columns (h dropped into the mantissa of 2^7), negated by the sign bit
      const float2 mhv = make_float2(__uint_as_float(__byte_perm(h[j >> 1], 0xC3000000u, 0x7610)),
                                     __uint_as_float(__byte_perm(h[j >> 1], 0xC3000000u, 0x7632)));
      const float2 t = mul2(make_float2(w[j], w[j + 1]), inv2);
      float2 y;                                             // kMagic + ceil(t - h / 65536) + z, per lane
      {
        const float2 u = add2(t, mhv);
        asm("add.rp.f32x2 %0, %1, %2;"
            : "=l"(*reinterpret_cast<uint64_t*>(&y))
            : "l"(*reinterpret_cast<const uint64_t*>(&u)), "l"(*reinterpret_cast<const uint64_t*>(&mz2)));
      }
      code[j] = __float_as_int(y.x) - 0x4B400000;           // may be -129 or 128: the pack saturates
      code[j + 1] = __float_as_int(y.y) - 0x4B400000;
    }
    uint32_t o[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) o[k] = pack_sat_s8x4(code[4 * k], code[4 * k + 1], code[4 * k + 2], code[4 * k + 3]);
    return make_uint4(o[0], o[1], o[2], o[3]);
  }
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const float t = __fmul_rn(w[j], gp.inv);
    if (FAST) {
      // 128 + h / 65536: h dropped into the mantissa of 2^7
      const float hv = __uint_as_float(__byte_perm(h[j >> 1], 0x43000000u, (j & 1) ? 0x7632 : 0x7610));
      const float y = __fadd_ru(__fsub_rn(t, hv), mz);       // kMagic + ceil(t - h / 65536) + z
      code[j] = __float_as_int(y) - 0x4B400000;               // may be -129 or 128: the pack saturates
    } else {
      const float hf = (float)((h[j >> 1] >> (16 * (j & 1))) & 0xFFFFu);
      const float f = floorf(t);
      const float up = (__fmul_rn(__fsub_rn(t, f), 65536.0f) > hf) ? 1.0f : 0.0f;
      const float qv = fminf(fmaxf(__fadd_rn(__fadd_rn(f, up), gp.z), -128.0f), 127.0f);
      code[j] = (int)qv;
    }
  }
  uint32_t o[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) o[k] = pack_sat_s8x4(code[4 * k], code[4 * k + 1], code[4 * k + 2], code[4 * k + 3]);
  return make_uint4(o[0], o[1], o[2], o[3]);
}

template <bool SINGLE, int CTAS>
__global__ void __launch_bounds__(K2Smem::kThreads, 1)
backproject_sr_kernel(const __grid_constant__ TcProblem single, const TcProblem* __restrict__ table,
                      const TileSchedule sched, int total_tiles, const StepScalars sc, int32_t* __restrict__ status) {
  static_assert(CTAS == 1 || !SINGLE, "CTA pairs run from a plan only");
  using S = typename std::conditional<CTAS == 2, K2PairSmem, K2Smem>::type;
  const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0u;   // 0 = the pair's leader, which issues the MMAs
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stage_base = smem;
  uint8_t* code_base = smem + S::kStages * S::kStageBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::kBarOffset);
  uint64_t* full = bars;
  uint64_t* empty = bars + S::kStages;
  uint64_t* acc_full = bars + 2 * S::kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* code_full = acc_empty + 2;
  uint64_t* code_empty = code_full + S::kCodeBufs;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(code_empty + S::kCodeBufs);
  float2* part = reinterpret_cast<float2*>(smem + S::kPartOffset);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const TcProblem* probs = SINGLE ? &single : table;

  if (threadIdx.x == 0) {
    for (int i = 0; i < S::kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], CTAS * S::kGroupWarps); }
    for (int i = 0; i < S::kCodeBufs; ++i) { mbar_init(&code_full[i], 1); mbar_init(&code_empty[i], 1); }
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    if (CTAS == 2) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
    else { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (CTAS == 2) cluster_sync_all();              // the peer's barriers exist before anything signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // tile -> (m block, n block) of its problem; consecutive tiles share the n block of N_b.  A pair takes two
  // adjacent m blocks, this CTA the one of its rank; the leader's `full` barriers count the loads of both CTAs
  // and its `acc_empty` barriers the epilogue warps of both.

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (TileWalk<SINGLE> tw(sched, total_tiles); ok && tw.valid(); tw.advance(), ++tcount) {
        const int2 item = tw.cur();
        const TcProblem* p = probs + item.x;
        const int local = item.y, mblocks = CTAS == 2 ? p->k2_mpairs : p->k2_mblocks;
        const int m0 = (local % mblocks) * (CTAS * kTileM) + (int)rank * kTileM, n0 = (local / mblocks) * S::kBN;
        const CUtensorMap* mapPk = &p->mapPk;
        const CUtensorMap* mapN3 = CTAS == 2 ? &p->mapN3h : &p->mapN3;
        const int kblocks = (p->r + kBK - 1) / kBK;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          if (!mbar_wait(&empty[s], ((it / S::kStages) & 1) ^ 1)) { ok = false; break; }
          uint8_t* sA = stage_base + s * S::kStageBytes;
          uint8_t* sB = sA + S::kABytes;
          if (CTAS == 2) {
            if (rank == 0) mbar_arrive_expect_tx(&full[s], 2 * S::kStageBytes);
            const uint32_t lead_full = mapa_u32(smem_u32(&full[s]), 0);
            tma_load_2d_pair(sA, mapPk, lead_full, kb * kBK, m0);
            tma_load_3d_pair(sB, mapN3, lead_full, 0, kb * kBK, n0 / 64 + 2 * (int)rank);
          } else if (p->right) {
            // D = N_b^T Q~^T: rows m0.. of N_b^T are columns of N_b (an MN-major A tile, two 64-row chunks),
            // columns n0.. of Q~^T are rows of Q~ (a K-major B tile of 256 rows)
            mbar_arrive_expect_tx(&full[s], S::kStageBytes);
            tma_load_3d(sA, &p->mapN3h, &full[s], 0, kb * kBK, m0 / 64);
            tma_load_2d(sB, &p->mapQk, &full[s], kb * kBK, n0);
          } else {
            mbar_arrive_expect_tx(&full[s], S::kStageBytes);
            tma_load_2d(sA, mapPk, &full[s], kb * kBK, m0);
            tma_load_3d(sB, mapN3, &full[s], 0, kb * kBK, n0 / 64);
          }
        }
      }
      if (!ok) raise_wait_expired(status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc_left = umma_idesc_bf16(CTAS * kTileM, S::kBN, false, true);
      constexpr uint32_t idesc_right = umma_idesc_bf16(CTAS * kTileM, S::kBN, true, false);
      const uint64_t desc_a0 = umma_smem_desc_sw128(smem_u32(stage_base), 16, 1024);
      const uint64_t desc_b0 = umma_smem_desc_sw128(smem_u32(stage_base) + S::kABytes, kBoxBytes, 1024);
      // right projection: A is MN-major (64-row chunks of 8 KB), B is K-major
      const uint64_t desc_am0 = umma_smem_desc_sw128(smem_u32(stage_base), kBoxBytes, 1024);
      const uint64_t desc_bk0 = umma_smem_desc_sw128(smem_u32(stage_base) + S::kABytes, 16, 1024);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (TileWalk<SINGLE> tw(sched, total_tiles); ok && tw.valid(); tw.advance(), ++tcount) {
        const TcProblem* p = probs + tw.cur().x;
        const int kblocks = (p->r + kBK - 1) / kBK;
        const bool right = p->right != 0;
        const uint32_t idesc = right ? idesc_right : idesc_left;
        const uint64_t astep = right ? (2048 >> 4) : (32 >> 4), bstep = right ? (32 >> 4) : (2048 >> 4);
        const uint32_t ab = tcount & 1;
        if (!(CTAS == 2 ? mbar_wait_cluster(&acc_empty[ab], ((tcount >> 1) & 1) ^ 1)
                        : mbar_wait(&acc_empty[ab], ((tcount >> 1) & 1) ^ 1))) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + ab * S::kBN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          if (!(CTAS == 2 ? mbar_wait_cluster(&full[s], (it / S::kStages) & 1) : mbar_wait(&full[s], (it / S::kStages) & 1))) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          // A is K-major (rows of 128 bytes, 16 K indices = 32 bytes further along the row),
          // B is MN-major (16 K indices = two 8-index groups of 1024 bytes)
          const uint64_t da = (right ? desc_am0 : desc_a0) + (uint64_t)((s * S::kStageBytes) >> 4);
          const uint64_t db = (right ? desc_bk0 : desc_b0) + (uint64_t)((s * S::kStageBytes) >> 4);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            if (CTAS == 2) umma_bf16_pair(d_tmem, da + k * astep, db + k * bstep, idesc, (kb | k) != 0);
            else umma_bf16(d_tmem, da + k * astep, db + k * bstep, idesc, (kb | k) != 0);
          }
          if (CTAS == 2) umma_commit_pair(&empty[s]); else umma_commit(&empty[s]);
        }
        if (ok) { if (CTAS == 2) umma_commit_pair(&acc_full[ab]); else umma_commit(&acc_full[ab]); }
      }
      if (!ok) raise_wait_expired(status);
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    // Sixteen warps in two groups of eight; group g takes the tiles whose accumulator buffer is g, so the
    // two groups work on different tiles and one fills the other's waits (scale loads, barriers, the
    // hand-over to the TMA store).  Within a group, warp (quarter q, slice sl) owns accumulator rows
    // 32q..32q+31 and columns 128*sl..128*sl+127; a row of the tile is one quantization group, so two threads
    // share a group and combine their minima and maxima through shared memory.  The pre-rounding weights
    // are written back over the accumulator in tensor memory between the two passes (registers are the
    // scarce resource with 18 warps on the SM: 5 warps share one 16K-register scheduler partition).
    const int grp = (warp - 2) >> 3;
    const int q = warp & 3, sl = ((warp - 2) >> 2) & 1;
    const int row = q * 32 + lane;
    const bool elected = (threadIdx.x == 64 + grp * S::kGroupThreads);
    const int bar_id = 1 + grp;
    const bool no_wd = (sc.lr_wd == 0.0f);
    const bool nearest = (sc.rounding == QG_ROUND_NEAREST);
    float2* gpart = part + grp * 2 * kTileM;
    uint8_t* cbuf = code_base + grp * S::kCodeBytes;   // the group's own buffer for the INT8 codes of its tile
    // the codes of a tile are fetched by the group itself: the first tile here, each later one as soon as
    // the previous tile's codes have been consumed (after pass 1), so the fetch overlaps pass 2
    auto fetch_codes = [&](int2 it2) {
      const TcProblem* p2 = probs + it2.x;
      const int mb2 = CTAS == 2 ? p2->k2_mpairs : p2->k2_mblocks;
      const int m2 = (it2.y % mb2) * (CTAS * kTileM) + (int)rank * kTileM, n2 = (it2.y / mb2) * S::kBN;
      mbar_arrive_expect_tx(&code_full[grp], S::kCodeBytes);
      tma_load_2d(cbuf, &p2->mapW, &code_full[grp], n2, m2);
      tma_load_2d(cbuf + S::kCodeBytes / 2, &p2->mapW, &code_full[grp], n2 + 128, m2);
    };
    {
      TileWalk<SINGLE> first(sched, total_tiles);
      if (grp == 1) first.advance();
      if (elected && first.valid()) fetch_codes(first.cur());
    }
    uint32_t tcount = 0;
    bool ok = true;
    for (TileWalk<SINGLE> tw(sched, total_tiles); ok && tw.valid(); tw.advance(), ++tcount) {
      if ((int)(tcount & 1) != grp) continue;
      const int2 item = tw.cur();
      const TcProblem* p = probs + item.x;
      const int local = item.y, mblocks = CTAS == 2 ? p->k2_mpairs : p->k2_mblocks;
      const int m0 = (local % mblocks) * (CTAS * kTileM) + (int)rank * kTileM, nblk = local / mblocks, n0 = nblk * S::kBN;
      const int pn = p->n, ngroups = p->ngroups;
      const int gi = m0 + row;                       // global row
      const bool row_ok = gi < p->m;
      const int ncols = min(S::kBN, pn - n0);        // valid columns of this (possibly ragged) group
      const int64_t ldw = p->ldw;
      float* g_scale = p->w_scales + (int64_t)gi * ngroups + nblk;
      float* g_zero = p->w_zeros + (int64_t)gi * ngroups + nblk;
      int8_t* g_codes = p->w_codes + (int64_t)gi * ldw;
      float* dbgW = p->dbgW ? p->dbgW + (int64_t)gi * ldw : nullptr;
      const uint32_t seed_lo = p->seed_lo, seed_hi = p->seed_hi;
      float s_old = 1.f, z_old = 0.f;
      if (row_ok) { s_old = __ldg(g_scale); z_old = __ldg(g_zero); }
      const uint32_t ab = tcount & 1;                // == grp: a group always drains the same accumulator buffer
      ok = mbar_wait(&code_full[grp], (tcount >> 1) & 1) && mbar_wait(&acc_full[ab], (tcount >> 1) & 1);
      ok = named_bar_and(bar_id, S::kGroupThreads, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + ab * S::kBN + sl * 128;
      // codes of columns 16*k16 .. +15 of this row: box (k16 / 8), 16-byte chunk (k16 % 8) ^ (row % 8)
      auto code_ptr = [&](int k16) -> uint4* {
        return reinterpret_cast<uint4*>(cbuf + (k16 >> 3) * (S::kCodeBytes / 2) + row * 128 + (((k16 & 7) ^ (row & 7)) << 4));
      };

      // ---- pass 1: W' of the thread's 128 columns, written back over the accumulator; minimum and maximum.
      // Pieces of 16 columns, the tensor-memory load of the next piece in flight while one is computed.
      const bool fast_dq = __all_sync(0xFFFFFFFFu, fabsf(z_old) <= 4.0e6f);
      const int myc0 = sl * 128;
      float mn = INFINITY, mx = -INFINITY;
      auto pass1_piece = [&](int pc, const uint32_t* acc) {
        float w[16];
        const uint4 cw = *code_ptr(sl * 8 + pc);
        if (fast_dq && no_wd) weights16<true, true>(cw, acc, z_old, s_old, sc.lr_alpha, 0.f, w);
        else if (fast_dq) weights16<true, false>(cw, acc, z_old, s_old, sc.lr_alpha, sc.lr_wd, w);
        else weights16<false, false>(cw, acc, z_old, s_old, sc.lr_alpha, sc.lr_wd, w);
        if (myc0 + 16 * pc + 16 <= ncols) {
#pragma unroll
          for (int i = 0; i < 16; i += 2) { mn = min3(mn, w[i], w[i + 1]); mx = max3(mx, w[i], w[i + 1]); }
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i)
            if (myc0 + 16 * pc + i < ncols) { mn = fminf(mn, w[i]); mx = fmaxf(mx, w[i]); }
        }
        uint32_t wb[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) wb[i] = __float_as_uint(w[i]);
        tmem_st_32x16(tacc + 16 * pc, wb);
      };
      {
        uint32_t a0[16], a1[16];
        tmem_ld_32x16(tacc, a0);
        tmem_ld_wait();
#pragma unroll 1
        for (int pc = 0; pc < 8; pc += 2) {
          tmem_ld_32x16(tacc + 16 * (pc + 1), a1);
          pass1_piece(pc, a0);
          tmem_ld_wait();
          if (pc + 2 < 8) tmem_ld_32x16(tacc + 16 * (pc + 2), a0);
          pass1_piece(pc + 1, a1);
          tmem_ld_wait();
        }
      }
      tmem_st_wait();
      gpart[sl * kTileM + row] = make_float2(mn, mx);
      fence_proxy_async_smem();                         // the old codes have been read: the buffer may be refilled
      named_bar_sync(bar_id, S::kGroupThreads);
      if (elected) {
        TileWalk<SINGLE> nx = tw;
        nx.advance();
        if (nx.valid()) { nx.advance(); if (nx.valid()) fetch_codes(nx.cur()); }
      }
      {
        const float2 pm = gpart[(sl ^ 1) * kTileM + row];
        mn = fminf(mn, pm.x);
        mx = fmaxf(mx, pm.y);
      }
      const GroupParams gp = group_params<8>(mn, mx);
      if (row_ok && sl == 0) { *g_scale = gp.s; *g_zero = gp.z; }

      // ---- pass 2: stochastic rounding to the new grid, codes written over the old ones in shared memory
      const bool fast_sr = __all_sync(0xFFFFFFFFu, fabsf(gp.z) <= 1024.0f);
      uint32_t kx[10], ky[10];
#pragma unroll
      for (int i = 0; i < 10; ++i) { kx[i] = seed_lo + (uint32_t)i * 0x9E3779B9u; ky[i] = seed_hi + (uint32_t)i * 0xBB67AE85u; }
      auto pass2_piece = [&](int pc, const uint32_t* wbits) {
        const int col = n0 + myc0 + 16 * pc;
        const float* w = reinterpret_cast<const float*>(wbits);
        uint4 out;
        if (nearest) {
          out = fast_sr ? rtn_codes16<true>(w, gp) : rtn_codes16<false>(w, gp);
        } else {
          const uint4 x0 = philox_rounds(make_uint4((uint32_t)(col >> 3), (uint32_t)gi, sc.step_lo, sc.step_hi), kx, ky);
          const uint4 x1 = philox_rounds(make_uint4((uint32_t)(col >> 3) + 1u, (uint32_t)gi, sc.step_lo, sc.step_hi), kx, ky);
          const uint32_t h[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
          out = fast_sr ? sr_codes16<true>(w, gp, h) : sr_codes16<false>(w, gp, h);
        }
        // sixteen new codes of this row, straight to global memory (the two halves of a 32-byte sector are
        // written by consecutive pieces and merge in L2); the ragged end of a row byte by byte
        if (row_ok && col + 16 <= pn) {
          *reinterpret_cast<uint4*>(g_codes + col) = out;
        } else if (row_ok && col < pn) {
          const uint32_t o4[4] = {out.x, out.y, out.z, out.w};
#pragma unroll
          for (int e = 0; e < 15; ++e)
            if (col + e < pn) g_codes[col + e] = (int8_t)((o4[e >> 2] >> (8 * (e & 3))) & 0xFFu);
        }
        if (dbgW != nullptr && row_ok) {
#pragma unroll
          for (int e = 0; e < 16; ++e)
            if (col + e < pn) dbgW[col + e] = w[e];
        }
      };
      {
        uint32_t a0[16], a1[16];
        tmem_ld_32x16(tacc, a0);
        tmem_ld_wait();
#pragma unroll 1
        for (int pc = 0; pc < 8; pc += 2) {
          tmem_ld_32x16(tacc + 16 * (pc + 1), a1);
          pass2_piece(pc, a0);
          tmem_ld_wait();
          if (pc + 2 < 8) {
            tmem_ld_32x16(tacc + 16 * (pc + 2), a0);
          } else {                                      // every read of this accumulator buffer has landed
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
              if (CTAS == 2) mbar_arrive_cluster(mapa_u32(smem_u32(&acc_empty[ab]), 0));
              else mbar_arrive(&acc_empty[ab]);
            }
          }
          pass2_piece(pc + 1, a1);
          tmem_ld_wait();
        }
      }

    }
    if (!ok && lane == 0) raise_wait_expired(status);
  }

  tc_fence_before_sync();
  __syncthreads();
  if (CTAS == 2) cluster_sync_all();              // neither CTA leaves while the other may still signal it
  if (warp == 1) {
    tc_fence_after_sync();
    if (CTAS == 2) tmem_dealloc_pair(tmem_base, 512); else tmem_dealloc(tmem_base, 512);
  }
}

// ============================================================================================
// host side
// ============================================================================================
// Scratch of one matrix: P~ (bf16, m x r, pitch r) then N_b (bf16, r x ldn).
struct TcScratch {
  uint16_t* Pt;
  uint16_t* Nb;
  int64_t ldn;
};

size_t scratch_pt_bytes(int64_t m, int64_t r) { return (size_t)round_up(m * r * 2, 1024); }
size_t scratch_nb_bytes(int64_t n, int64_t r) { return (size_t)round_up(r * round_up(n, 64) * 2, 1024); }

TcScratch carve(void* base, int64_t m, int64_t n, int64_t r) {
  TcScratch w;
  w.Pt = reinterpret_cast<uint16_t*>(base);
  w.Nb = reinterpret_cast<uint16_t*>(reinterpret_cast<char*>(base) + scratch_pt_bytes(m, r));
  w.ldn = round_up(n, 64);
  return w;
}

// Extents as the projection kernel sees them: rows of the projection matrix (its K extent) and columns of the
// low-rank state.  Left: (m, n).  Right: (n, m).
inline int64_t proj_rows(const StepArgs& a) { return a.right ? a.n : a.m; }
inline int64_t state_cols(const StepArgs& a) { return a.right ? a.m : a.n; }

// 1: the projection kernel converts the INT4 codes of P itself (converter warps); 0 (the default): P is
// dequantized to bf16 by a separate grouped launch first.  Both give the same results bit for bit; measured on
// B200 the separate launch is the faster arrangement (see the note at the converter warps).
int g_fuse_dequant = 0;

// The projection kernel converts the INT4 codes of P itself when a 128-wide rank block is whole and lies inside
// one quantization group; other code widths (the ablation) and ragged ranks take the bf16 copy made beforehand.
inline bool fused_dequant(const StepArgs& a) { return g_fuse_dequant && a.P.bits == 4 && a.r % kTileM == 0; }

int fill_problem(const StepArgs& a, const TcScratch& w, TcProblem* p, int bn) {
  memset(p, 0, sizeof(*p));
  bool ok = true;
  const int64_t prow = proj_rows(a), scol = state_cols(a);
  ok &= make_map(&p->mapP, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, w.Pt, a.r, prow, a.r, 64, kBK, CU_TENSOR_MAP_SWIZZLE_128B);
  ok &= make_map(&p->mapG, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.G, a.n, a.m, a.ldg, 64, kBK, CU_TENSOR_MAP_SWIZZLE_128B);
  ok &= make_map(&p->mapPk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, w.Pt, a.r, prow, a.r, 64, kTileM, CU_TENSOR_MAP_SWIZZLE_128B);
  const int64_t r_whole = a.r & ~int64_t(63), n_whole = a.n & ~int64_t(63);
  ok &= make_map_chunked(&p->mapP3, w.Pt, prow, r_whole > 0 ? r_whole / 64 : 1, a.r, kBK, 2);
  ok &= make_map_chunked(&p->mapG3, a.G, a.m, n_whole > 0 ? n_whole / 64 : 1, a.ldg, kBK, bn / 64);
  ok &= make_map_chunked(&p->mapG3h, a.G, a.m, n_whole > 0 ? n_whole / 64 : 1, a.ldg, kBK, 2);
  ok &= make_map_chunked(&p->mapN3, w.Nb, a.r, w.ldn / 64, w.ldn, kBK, 4);
  ok &= make_map_chunked(&p->mapN3h, w.Nb, a.r, w.ldn / 64, w.ldn, kBK, 2);
  // right projection: G (inner n = K, outer m) in boxes of 64 x 128 rows, Q~ (inner r = K, outer n) in 64 x 256
  ok &= make_map(&p->mapGk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.G, a.n, a.m, a.ldg, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
  ok &= make_map(&p->mapQk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, w.Pt, a.r, prow, a.r, 64, 256, CU_TENSOR_MAP_SWIZZLE_128B);
  p->r_whole = (int32_t)r_whole;
  p->n_whole = (int32_t)n_whole;
  p->p_codes = reinterpret_cast<const uint8_t*>(a.P.codes);
  p->p_scales = a.P.scales;
  p->p_zeros = a.P.zeros;
  p->pt = w.Pt;
  p->p_row_bytes = a.P.ld / 2;
  p->p_ngroups = (int32_t)ceil_div(a.r, kGroup);
  p->fuse_a = fused_dequant(a) ? 1 : 0;
  ok &= make_map(&p->mapW, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.W.codes, a.n, a.m, a.W.ld, 128, kTileM,
                 CU_TENSOR_MAP_SWIZZLE_128B);
  if (a.state8) {
    ok &= make_map(&p->mapM, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.M, scol, a.r, a.ldmv, kChunk, 32, CU_TENSOR_MAP_SWIZZLE_NONE);
    ok &= make_map(&p->mapV, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.V, scol, a.r, a.ldmv, kChunk, 32, CU_TENSOR_MAP_SWIZZLE_NONE);
  } else {
    ok &= make_map(&p->mapM, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.M, scol, a.r, a.ldmv, kChunk, 16, CU_TENSOR_MAP_SWIZZLE_128B);
    ok &= make_map(&p->mapV, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.V, scol, a.r, a.ldmv, kChunk, 16, CU_TENSOR_MAP_SWIZZLE_128B);
  }
  if (!ok) {
    note_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled");
    return QG_CUDA_ERROR;
  }
  p->M = a.M; p->V = a.V; p->w_codes = reinterpret_cast<int8_t*>(a.W.codes);
  p->w_scales = a.W.scales;
  p->w_zeros = a.W.zeros;
  p->dbgR = a.dbg.R; p->dbgN = a.dbg.N; p->dbgW = a.dbg.W_pre; p->dbgNb = a.dbg.N_b;
  p->nb = w.Nb;
  p->ldmv = a.ldmv; p->ldw = a.W.ld; p->ldn = w.ldn;
  p->m = (int32_t)a.m; p->n = (int32_t)a.n; p->r = (int32_t)a.r;
  p->right = a.right ? 1 : 0; p->k1_k = (int32_t)prow; p->k1_n = (int32_t)scol;
  p->state8 = a.state8 ? 1 : 0; p->nsb = (int32_t)ceil_div(scol, 32); p->m_scale = a.M_scale; p->v_scale = a.V_scale;
  p->ngroups = (int32_t)ceil_div(a.n, kGroup);
  p->seed_lo = a.sc.seed_lo; p->seed_hi = a.sc.seed_hi;
  p->k1_rblocks = (int32_t)ceil_div(a.r, kTileM);
  p->k1_tiles = p->k1_rblocks * (int32_t)ceil_div(scol, bn);
  p->k1_rpairs = (p->k1_rblocks + 1) / 2;
  p->k1p_tiles = p->k1_rpairs * (int32_t)ceil_div(scol, 256);
  p->k2_mblocks = (int32_t)ceil_div(a.m, kTileM);
  p->k2_tiles = p->k2_mblocks * (int32_t)ceil_div(a.n, K2Smem::kBN);
  p->k2_mpairs = (p->k2_mblocks + 1) / 2;
  p->k2p_tiles = p->k2_mpairs * (int32_t)ceil_div(a.n, K2Smem::kBN);
  return QG_OK;
}

int sm_count() {
  static int n = [] {
    int dev = 0, v = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    return v > 0 ? v : 148;
  }();
  return n;
}

// Opts a kernel instance into its dynamic shared memory, once per device and instance (`done` is the calling
// launcher's own flag array, one launcher per instance).
template <class K>
int set_smem_once(K kernel, int bytes, bool* done) {
  int dev = 0;
  QG_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return QG_UNSUPPORTED_SHAPE;
  if (done[dev]) return QG_OK;
  QG_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  done[dev] = true;
  return QG_OK;
}

// The projection's column-tile width: 256 halves the operand traffic per flop of the 128-wide tile,
// but only pays once there are enough tiles to occupy every SM.
int choose_bn(int64_t tiles_at_256) { return tiles_at_256 >= 2 * (int64_t)sm_count() ? 256 : 128; }

template <int BN, bool SINGLE, int CTAS, bool S8 = false, int MVS = 0>
int launch_k1(const TcProblem* single, const TcProblem* table, const TileSchedule& sched, int grid_planned,
              int total_tiles, const StepScalars& sc, int32_t* status, cudaStream_t st, int conv_active) {
  using S = K1Smem<BN, CTAS, MVS>;
  auto kern = project_adam_kernel<BN, SINGLE, CTAS, S8, MVS>;
  static bool smem_set[64] = {};
  int rc = set_smem_once(kern, S::kBytes, smem_set);
  if (rc != QG_OK) return rc;
  const int sms = sm_count();
  const int grid = SINGLE ? (total_tiles < sms ? total_tiles : sms) : grid_planned;
  static const TcProblem dummy{};
  if (CTAS == 1) {
    kern<<<grid, S::kThreads, S::kBytes, st>>>(single ? *single : dummy, table, sched, total_tiles, sc, status, conv_active);
  } else {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(S::kThreads);
    cfg.dynamicSmemBytes = S::kBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    QG_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, dummy, table, sched, total_tiles, sc, status, conv_active));
  }
  QG_LAUNCH_CHECK();
  return QG_OK;
}

template <bool SINGLE, int CTAS>
int launch_k2(const TcProblem* single, const TcProblem* table, const TileSchedule& sched, int grid_planned,
              int total_tiles, const StepScalars& sc, int32_t* status, cudaStream_t st) {
  using S = typename std::conditional<CTAS == 2, K2PairSmem, K2Smem>::type;
  auto kern = backproject_sr_kernel<SINGLE, CTAS>;
  static bool smem_set[64] = {};
  int rc = set_smem_once(kern, S::kBytes, smem_set);
  if (rc != QG_OK) return rc;
  const int sms = sm_count();
  const int grid = SINGLE ? (total_tiles < sms ? total_tiles : sms) : grid_planned;
  static const TcProblem dummy{};
  if (CTAS == 1) {
    kern<<<grid, S::kThreads, S::kBytes, st>>>(single ? *single : dummy, table, sched, total_tiles, sc, status);
  } else {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(S::kThreads);
    cfg.dynamicSmemBytes = S::kBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    QG_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, dummy, table, sched, total_tiles, sc, status));
  }
  QG_LAUNCH_CHECK();
  return QG_OK;
}

// ---- P~ = bf16(dequant(P)) for a list of matrices in one launch
struct DequantItem {
  qg_qtensor P;
  uint16_t* out;
  int32_t block0, nblocks;   // blocks of 256 threads; a block converts kDqUnits * 256 units of 8 columns
};

// Eight consecutive columns of a row: one 32-bit word of INT4 codes -> 16 bytes of bf16((q - z) * s).  FAST: the
// stored nibble (code + 8) is dropped into the mantissa of 2^23 and (2^23 + 8 + z) subtracted, which gives q - z
// exactly without an integer-to-float conversion (|z| < 2^22).
template <bool FAST>
__device__ __forceinline__ uint4 dequant8_int4(uint32_t w, float s, float z) {
  const float c = 8388616.0f + z;
  const float2 mc = make_float2(-c, -c), s2 = make_float2(s, s);
  const uint32_t lo4 = w & 0x0F0F0F0Fu, hi4 = (w >> 4) & 0x0F0F0F0Fu;   // even and odd columns, one per byte
  uint32_t o[4];
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    float2 v;
    if (FAST) {
      v = mul2(add2(make_float2(__uint_as_float(__byte_perm(lo4, 0x4B000000u, 0x7650 + b)),
                                __uint_as_float(__byte_perm(hi4, 0x4B000000u, 0x7650 + b))), mc), s2);
    } else {
      v.x = __fmul_rn(__fsub_rn((float)((int)((lo4 >> (8 * b)) & 0xFu) - 8), z), s);
      v.y = __fmul_rn(__fsub_rn((float)((int)((hi4 >> (8 * b)) & 0xFu) - 8), z), s);
    }
    const __nv_bfloat162 h2 = __floats2bfloat162_rn(v.x, v.y);
    o[b] = *reinterpret_cast<const uint32_t*>(&h2);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}

// The unit of work is eight columns.  A block converts kDqUnits * 256 consecutive units; a thread takes kDqUnits of
// them, 256 units apart, so that a warp reads 128 contiguous bytes of codes and writes 512 contiguous bytes of
// bf16 per step, and has all its loads in flight before it converts the first.
constexpr int kDqUnits = 8;

__global__ void __launch_bounds__(256)
dequant_p_grouped_kernel(const DequantItem* __restrict__ items, const int32_t* __restrict__ block_item) {
  const DequantItem& it = items[__ldg(block_item + blockIdx.x)];   // host-made map: block -> matrix of the chunk
  const uint32_t cols = (uint32_t)it.P.cols, rows = (uint32_t)it.P.rows;
  const uint32_t per_row = cols / 8, ngroups = (cols + kGroup - 1) / kGroup, total = rows * per_row;   // r % 32 == 0
  const uint32_t base = (blockIdx.x - (uint32_t)it.block0) * (kDqUnits * 256u) + threadIdx.x;
  if (it.P.bits != 4) {                              // the 2- and 8-bit projections of the ablation: plain conversion
    for (int u = 0; u < kDqUnits; ++u) {
      const uint32_t idx = base + 256u * u;
      if (idx >= total) break;
      const uint32_t row = idx / per_row, c0 = (idx - row * per_row) * 8;
      const uint32_t g = c0 / kGroup;
      const float s = __ldg(it.P.scales + (size_t)row * ngroups + g), z = __ldg(it.P.zeros + (size_t)row * ngroups + g);
      float q[8], v[8];
      load_codes8(it.P, row, c0, 8, q);
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = __fmul_rn(__fsub_rn(q[e], z), s);
      *reinterpret_cast<uint4*>(it.out + (size_t)row * cols + c0) = pack_bf16x8(v);
    }
    return;
  }
  uint32_t w[kDqUnits];
  float s[kDqUnits], z[kDqUnits];
  uint4* out[kDqUnits];
  const uint32_t row_bytes = (uint32_t)(it.P.ld / 2);
#pragma unroll
  for (int u = 0; u < kDqUnits; ++u) {
    const uint32_t idx = base + 256u * u;
    out[u] = nullptr;
    if (idx >= total) continue;
    const uint32_t row = idx / per_row, c0 = (idx - row * per_row) * 8;
    const uint32_t g = c0 / kGroup;
    w[u] = __ldcs(reinterpret_cast<const uint32_t*>((const uint8_t*)it.P.codes + (size_t)row * row_bytes + (c0 >> 1)));
    s[u] = __ldg(it.P.scales + (size_t)row * ngroups + g);
    z[u] = __ldg(it.P.zeros + (size_t)row * ngroups + g);
    out[u] = reinterpret_cast<uint4*>(it.out + (size_t)row * cols + c0);
  }
#pragma unroll
  for (int u = 0; u < kDqUnits; ++u) {
    // a warp-uniform choice (every lane votes, also those past the end), so that the plain form is a branch
    // not taken rather than work done and discarded
    const bool valid = out[u] != nullptr;
    if (__all_sync(0xFFFFFFFFu, !valid || fabsf(z[u]) < 4.0e6f)) {
      if (valid) *out[u] = dequant8_int4<true>(w[u], s[u], z[u]);
    } else {
      if (valid) *out[u] = dequant8_int4<false>(w[u], s[u], z[u]);
    }
  }
}

}  // namespace

// (m, n) here are the projection's row count and the state's column count: (m, n) of the matrix for the left
// form, (n, m) for the right one
size_t tc_workspace_bytes(int64_t m, int64_t n, int64_t r) { return scratch_pt_bytes(m, r) + scratch_nb_bytes(n, r); }

int launch_project_step_tc(const StepArgs& a, cudaStream_t st) {
  const TcScratch w = carve(a.ws, proj_rows(a), state_cols(a), a.r);
  int rc = fused_dequant(a) ? QG_OK : launch_dequant_p(a.P, w.Pt, a.r, st);
  if (rc != QG_OK) return rc;
  const int bn = choose_bn(ceil_div(a.r, kTileM) * ceil_div(state_cols(a), 256));
  TcProblem prob;
  rc = fill_problem(a, w, &prob, bn);
  if (rc != QG_OK) return rc;
  const TileSchedule none{nullptr, nullptr, 1};
  if (a.state8) {
    rc = bn == 256 ? launch_k1<256, true, 1, true>(&prob, nullptr, none, 0, prob.k1_tiles, a.sc, a.status, st, prob.fuse_a)
                   : launch_k1<128, true, 1, true>(&prob, nullptr, none, 0, prob.k1_tiles, a.sc, a.status, st, prob.fuse_a);
  } else {
    rc = bn == 256 ? launch_k1<256, true, 1>(&prob, nullptr, none, 0, prob.k1_tiles, a.sc, a.status, st, prob.fuse_a)
                   : launch_k1<128, true, 1>(&prob, nullptr, none, 0, prob.k1_tiles, a.sc, a.status, st, prob.fuse_a);
  }
  if (rc != QG_OK) return rc;
  return launch_k2<true, 1>(&prob, nullptr, none, 0, prob.k2_tiles, a.sc, a.status, st);
}

// ============================================================================================
// plans: a fixed list of matrices prepared once (tensor maps, tile tables) and stepped many times
// ============================================================================================
struct PlanChunk {
  int first, count;          // items [first, first + count)
  int k1_tiles, k2_tiles, k2p_tiles, bn;
  int dq_blocks;
  int k1_grid, k2_grid, pairs, k1_pairs, k1p_tiles, state8;
  int conv_active;           // some matrix of the chunk has its projection converted inside the projection kernel
  int k1_deep;               // long main loops (on average 48 K blocks or more per tile): five operand stages, two M/V slots
  size_t k1_start_off, k1_items_off, k2_start_off, k2_items_off;   // int32 offsets into the schedule buffer
  size_t dq_map_off;                                                // same: block -> item map of the dequantize launch
};

struct Plan {
  std::vector<PlanChunk> chunks;
  TcProblem* table_dev = nullptr;
  DequantItem* dq_dev = nullptr;
  int32_t* sched_dev = nullptr;
  int count = 0;
};

// Longest-processing-time-first assignment of tiles to `grid` CTAs: tiles in order of decreasing cost (ties
// keep their order, which keeps tiles that share an operand block next to each other), each to the CTA with
// the least work so far.  Appends start[grid + 1] and the (problem, tile) pairs to `buf`.
void schedule_tiles(const std::vector<int2>& tiles, const std::vector<float>& cost, int grid, std::vector<int32_t>& buf,
                    size_t* start_off, size_t* items_off) {
  std::vector<int> order(tiles.size());
  for (size_t i = 0; i < order.size(); ++i) order[i] = (int)i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return cost[a] > cost[b]; });
  using Load = std::pair<float, int>;                         // (work so far, CTA)
  std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
  for (int c = 0; c < grid; ++c) heap.push({0.f, c});
  std::vector<std::vector<int>> per_cta((size_t)grid);
  for (int t : order) {
    Load l = heap.top();
    heap.pop();
    per_cta[(size_t)l.second].push_back(t);
    heap.push({l.first + cost[t], l.second});
  }
  *start_off = buf.size();
  int32_t run = 0;
  for (int c = 0; c < grid; ++c) { buf.push_back(run); run += (int32_t)per_cta[(size_t)c].size(); }
  buf.push_back(run);
  if (buf.size() & 1) buf.push_back(0);                      // int2 alignment of the pairs
  *items_off = buf.size();
  for (int c = 0; c < grid; ++c)
    for (int t : per_cta[(size_t)c]) { buf.push_back(tiles[t].x); buf.push_back(tiles[t].y); }
}

// bit 0: the back-projection of a plan runs as CTA pairs (cta_group::2); bit 1: the projection does; bit 2: the
// back-projection does where it pays, i.e. in chunks whose ranks average 1024 or more (measured on LLaMA-7B under
// the power cap: 13.9-14.2 ms against 15.1 unpaired, the halved operand traffic buys clock; on LLaMA-1B, r = 512,
// pairs are 3 % slower).  Read when a plan is created.
int g_pair_mode = 6;

// Scratch is shared by the matrices of a chunk; a chunk is a run of consecutive items whose P~ and N_b fit
// both the caller's workspace and this budget.  Few, long launches win: with two or three tiles per CTA the
// fill and drain of the software pipelines cost a third of a launch, which outweighs keeping N_b (written by
// the first kernel, read by the second) inside the 126 MB L2.
size_t g_chunk_budget = 256ull << 20;

size_t plan_table_bytes(const StepArgs* items, int32_t count) {
  size_t sched = 0;                                           // int32 words: pairs of every tile + starts per chunk
  for (int32_t i = 0; i < count; ++i) {
    const int64_t k1 = ceil_div(items[i].r, kTileM) * ceil_div(state_cols(items[i]), 128);
    const int64_t k2 = ceil_div(items[i].m, kTileM) * ceil_div(items[i].n, K2Smem::kBN);
    sched += (size_t)(2 * (k1 + k2)) + 2 * (size_t)(sm_count() + 3);
    sched += (size_t)ceil_div(proj_rows(items[i]) * (items[i].r / 32), 256) + 2;   // block -> matrix map of the dequantize launch
  }
  return (size_t)round_up((int64_t)count * sizeof(TcProblem), 256) + (size_t)round_up((int64_t)count * sizeof(DequantItem), 256) +
         sched * sizeof(int32_t) + 256;
}

int plan_create(const StepArgs* items, int32_t count, void* table_dev, size_t table_bytes, void* workspace,
                size_t workspace_bytes, Plan** out) {
  if (table_bytes < plan_table_bytes(items, count)) return QG_WORKSPACE_TOO_SMALL;
  std::vector<TcProblem> probs((size_t)count);
  std::vector<DequantItem> dq((size_t)count);
  std::vector<int32_t> sched;
  Plan* plan = new Plan();
  plan->count = count;
  const size_t budget = workspace_bytes < g_chunk_budget ? workspace_bytes : g_chunk_budget;
  int i = 0;
  while (i < count) {
    // extent of the chunk
    size_t used = 0;
    int j = i;
    int64_t tiles256 = 0;
    while (j < count) {
      const size_t need = tc_workspace_bytes(proj_rows(items[j]), state_cols(items[j]), items[j].r);
      if (need > workspace_bytes) { delete plan; return QG_WORKSPACE_TOO_SMALL; }
      if (j > i && used + need > budget) break;
      used += need;
      tiles256 += ceil_div(items[j].r, kTileM) * ceil_div(state_cols(items[j]), 256);
      ++j;
    }
    PlanChunk ch{};
    ch.first = i; ch.count = j - i;
    ch.bn = choose_bn(tiles256);
    // the projection runs as CTA pairs when asked to, on 256-column tiles, if every rank of the chunk fills
    // whole 256-row pairs
    ch.k1_pairs = (g_pair_mode & 2) && ch.bn == 256;
    for (int k = i; k < j && ch.k1_pairs; ++k)
      if (items[k].r % 256 != 0) ch.k1_pairs = 0;
    // the back-projection runs as CTA pairs when asked to, unless the chunk holds a right-hand item (the paired
    // kernel knows the left form only); decided here, before the tile lists are made, because the lists of the
    // two forms differ (tiles of 256 rows against tiles of 128)
    ch.pairs = g_pair_mode & 1;
    if (g_pair_mode & 4) {
      int64_t rsum = 0;
      for (int k = i; k < j; ++k) rsum += items[k].r;
      if (rsum >= (int64_t)1024 * (j - i)) ch.pairs = 1;
    }
    for (int k = i; k < j; ++k) {
      if (items[k].right) ch.pairs = 0;
      if (items[k].state8) ch.state8 = 1;
    }
    size_t off = 0;
    std::vector<int2> t1, t2;
    std::vector<float> c1, c2;
    std::vector<int32_t> dq_map;
    for (int k = i; k < j; ++k) {
      const StepArgs& a = items[k];
      const TcScratch w = carve(reinterpret_cast<char*>(workspace) + off, proj_rows(a), state_cols(a), a.r);
      off += tc_workspace_bytes(proj_rows(a), state_cols(a), a.r);
      const int rc = fill_problem(a, w, &probs[k], ch.bn);
      if (rc != QG_OK) { delete plan; return rc; }
      ch.k1_tiles += probs[k].k1_tiles;
      ch.k2_tiles += probs[k].k2_tiles;
      // cost of a tile in K blocks of its main loop, plus a constant for its epilogue and hand-over
      const int k1n = ch.k1_pairs ? probs[k].k1p_tiles : probs[k].k1_tiles;
      for (int t = 0; t < k1n; ++t) { t1.push_back(make_int2(k - i, t)); c1.push_back((float)ceil_div(proj_rows(a), kBK) + 6.f); }
      ch.k1p_tiles += probs[k].k1p_tiles;
      const int k2n = ch.pairs ? probs[k].k2p_tiles : probs[k].k2_tiles;
      for (int t = 0; t < k2n; ++t) { t2.push_back(make_int2(k - i, t)); c2.push_back((float)ceil_div(a.r, kBK) + 6.f); }
      ch.k2p_tiles += probs[k].k2p_tiles;
      dq[k].P = a.P; dq[k].out = w.Pt;
      dq[k].block0 = ch.dq_blocks;
      dq[k].nblocks = fused_dequant(a) ? 0 : (int32_t)ceil_div(proj_rows(a) * (a.r / 8), 256 * 8);
      if (fused_dequant(a)) ch.conv_active = 1;
      ch.dq_blocks += dq[k].nblocks;
      for (int32_t blk = 0; blk < dq[k].nblocks; ++blk) dq_map.push_back(k - i);
    }
    {
      double kb_sum = 0.0;
      for (float c : c1) kb_sum += (double)c - 6.0;
      ch.k1_deep = !c1.empty() && kb_sum / (double)c1.size() >= 48.0;
    }
    if (ch.k1_pairs) ch.k1_grid = 2 * (ch.k1p_tiles < sm_count() / 2 ? ch.k1p_tiles : sm_count() / 2);
    else ch.k1_grid = ch.k1_tiles < sm_count() ? ch.k1_tiles : sm_count();
    if (ch.pairs) ch.k2_grid = 2 * (ch.k2p_tiles < sm_count() / 2 ? ch.k2p_tiles : sm_count() / 2);   // CTA pairs
    else ch.k2_grid = ch.k2_tiles < sm_count() ? ch.k2_tiles : sm_count();
    schedule_tiles(t1, c1, ch.k1_pairs ? ch.k1_grid / 2 : ch.k1_grid, sched, &ch.k1_start_off, &ch.k1_items_off);
    if (sched.size() & 1) sched.push_back(0);
    schedule_tiles(t2, c2, ch.pairs ? ch.k2_grid / 2 : ch.k2_grid, sched, &ch.k2_start_off, &ch.k2_items_off);
    if (sched.size() & 1) sched.push_back(0);
    ch.dq_map_off = sched.size();
    sched.insert(sched.end(), dq_map.begin(), dq_map.end());
    if (sched.size() & 1) sched.push_back(0);
    plan->chunks.push_back(ch);
    i = j;
  }
  plan->table_dev = reinterpret_cast<TcProblem*>(table_dev);
  plan->dq_dev = reinterpret_cast<DequantItem*>(reinterpret_cast<char*>(table_dev) +
                                                round_up((int64_t)count * sizeof(TcProblem), 256));
  plan->sched_dev = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(plan->dq_dev) +
                                               round_up((int64_t)count * sizeof(DequantItem), 256));
  if (reinterpret_cast<char*>(plan->sched_dev + sched.size()) > reinterpret_cast<char*>(table_dev) + table_bytes) {
    delete plan;
    return QG_WORKSPACE_TOO_SMALL;
  }
  cudaError_t e = cudaMemcpy(plan->table_dev, probs.data(), (size_t)count * sizeof(TcProblem), cudaMemcpyHostToDevice);
  if (e == cudaSuccess)
    e = cudaMemcpy(plan->dq_dev, dq.data(), (size_t)count * sizeof(DequantItem), cudaMemcpyHostToDevice);
  if (e == cudaSuccess)
    e = cudaMemcpy(plan->sched_dev, sched.data(), sched.size() * sizeof(int32_t), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    note_cuda_error(e, "cudaMemcpy(plan table)");
    delete plan;
    return QG_CUDA_ERROR;
  }
  *out = plan;
  return QG_OK;
}

// One step of every chunk.  With `ev` (4 events per chunk, created by the caller) an event is recorded
// before the chunk's first kernel and after each of its three kernels.
int plan_step(const Plan* plan, const StepScalars& sc, int32_t* status, cudaStream_t st, cudaEvent_t* ev) {
  size_t c = 0;
  for (const PlanChunk& ch : plan->chunks) {
    if (ev) QG_CUDA_TRY(cudaEventRecord(ev[4 * c + 0], st));
    if (ch.dq_blocks > 0) {                              // matrices whose projection the first kernel does not convert itself
      dequant_p_grouped_kernel<<<ch.dq_blocks, 256, 0, st>>>(plan->dq_dev + ch.first, plan->sched_dev + ch.dq_map_off);
      QG_LAUNCH_CHECK();
    }
    if (ev) QG_CUDA_TRY(cudaEventRecord(ev[4 * c + 1], st));
    const TcProblem* tab = plan->table_dev + ch.first;
    const TileSchedule s1{plan->sched_dev + ch.k1_start_off, reinterpret_cast<const int2*>(plan->sched_dev + ch.k1_items_off),
                          ch.k1_pairs ? 2 : 1};
    const TileSchedule s2{plan->sched_dev + ch.k2_start_off, reinterpret_cast<const int2*>(plan->sched_dev + ch.k2_items_off),
                          ch.pairs ? 2 : 1};
    int rc;
    if (ch.state8) {       // some matrix of the chunk keeps its moments in 8 bits
      rc = ch.k1_pairs  ? launch_k1<256, false, 2, true>(nullptr, tab, s1, ch.k1_grid, ch.k1p_tiles, sc, status, st, ch.conv_active)
           : ch.bn == 256 ? launch_k1<256, false, 1, true>(nullptr, tab, s1, ch.k1_grid, ch.k1_tiles, sc, status, st, ch.conv_active)
                          : launch_k1<128, false, 1, true>(nullptr, tab, s1, ch.k1_grid, ch.k1_tiles, sc, status, st, ch.conv_active);
    } else {
      rc = (ch.k1_pairs && ch.k1_deep) ? launch_k1<256, false, 2, false, 2>(nullptr, tab, s1, ch.k1_grid, ch.k1p_tiles, sc, status, st, ch.conv_active)
           : ch.k1_pairs  ? launch_k1<256, false, 2>(nullptr, tab, s1, ch.k1_grid, ch.k1p_tiles, sc, status, st, ch.conv_active)
           : ch.bn == 256 ? launch_k1<256, false, 1>(nullptr, tab, s1, ch.k1_grid, ch.k1_tiles, sc, status, st, ch.conv_active)
                          : launch_k1<128, false, 1>(nullptr, tab, s1, ch.k1_grid, ch.k1_tiles, sc, status, st, ch.conv_active);
    }
    if (rc != QG_OK) return rc;
    if (ev) QG_CUDA_TRY(cudaEventRecord(ev[4 * c + 2], st));
    rc = ch.pairs ? launch_k2<false, 2>(nullptr, tab, s2, ch.k2_grid, ch.k2p_tiles, sc, status, st)
                  : launch_k2<false, 1>(nullptr, tab, s2, ch.k2_grid, ch.k2_tiles, sc, status, st);
    if (rc != QG_OK) return rc;
    if (ev) QG_CUDA_TRY(cudaEventRecord(ev[4 * c + 3], st));
    ++c;
  }
  return QG_OK;
}

// One step with an event pair around every launch; blocks until the step has finished.
// ms[0..2] receive the summed durations of the dequantize, projection and back-projection launches,
// launches[0..2] their counts.
int plan_step_timed(const Plan* plan, const StepScalars& sc, int32_t* status, cudaStream_t st, float* ms,
                    int32_t* launches) {
  const size_t nch = plan->chunks.size();
  std::vector<cudaEvent_t> ev(4 * nch, nullptr);
  int rc = QG_OK;
  for (auto& e : ev)
    if (cudaEventCreate(&e) != cudaSuccess) rc = QG_CUDA_ERROR;
  if (rc == QG_OK) rc = plan_step(plan, sc, status, st, ev.data());
  if (rc == QG_OK && cudaStreamSynchronize(st) != cudaSuccess) rc = QG_CUDA_ERROR;
  for (int k = 0; k < 3; ++k) { ms[k] = 0.f; launches[k] = 0; }
  if (rc == QG_OK) {
    for (size_t c = 0; c < nch; ++c)
      for (int k = 0; k < 3; ++k) {
        float t = 0.f;
        if (k == 0 && plan->chunks[c].dq_blocks == 0) continue;      // no dequantize launch in this chunk
        if (cudaEventElapsedTime(&t, ev[4 * c + k], ev[4 * c + k + 1]) == cudaSuccess) { ms[k] += t; launches[k] += 1; }
      }
  }
  for (auto& e : ev)
    if (e) cudaEventDestroy(e);
  (void)cudaGetLastError();
  return rc;
}

void plan_destroy(Plan* plan) { delete plan; }
int set_pair_mode(int mask) { g_pair_mode = mask & 7; return QG_OK; }
int set_fused_dequant(int on) { g_fuse_dequant = on ? 1 : 0; return QG_OK; }
int set_chunk_budget(size_t bytes) { g_chunk_budget = bytes; return QG_OK; }

// Registers, thread limit and shared memory of the tensor-core kernels as the loaded module reports them.
int tc_kernel_info(char* buf, size_t cap) {
  size_t used = 0;
  auto add = [&](const char* name, const void* fn, int threads, int dyn_smem) {
    cudaFuncAttributes at{};
    const cudaError_t e = cudaFuncGetAttributes(&at, fn);
    int n = 0;
    if (e != cudaSuccess) {
      n = snprintf(buf + used, cap - used, "%s: %s\n", name, cudaGetErrorName(e));
      (void)cudaGetLastError();
    } else {
      n = snprintf(buf + used, cap - used, "%s: regs %d, max threads %d, launched with %d threads, dynamic smem %d, static smem %zu, local %zu\n",
                   name, at.numRegs, at.maxThreadsPerBlock, threads, dyn_smem, at.sharedSizeBytes, at.localSizeBytes);
    }
    if (n > 0) used = (used + (size_t)n < cap) ? used + (size_t)n : cap - 1;
  };
  add("project_adam<128,single>", (const void*)project_adam_kernel<128, true, 1>, K1Smem<128>::kThreads, K1Smem<128>::kBytes);
  add("project_adam<256,single>", (const void*)project_adam_kernel<256, true, 1>, K1Smem<256>::kThreads, K1Smem<256>::kBytes);
  add("project_adam<128,table>", (const void*)project_adam_kernel<128, false, 1>, K1Smem<128>::kThreads, K1Smem<128>::kBytes);
  add("project_adam<256,table>", (const void*)project_adam_kernel<256, false, 1>, K1Smem<256>::kThreads, K1Smem<256>::kBytes);
  add("project_adam<256,table,pairs>", (const void*)project_adam_kernel<256, false, 2>, K1Smem<256, 2>::kThreads, K1Smem<256, 2>::kBytes);
  add("backproject_sr<single>", (const void*)backproject_sr_kernel<true, 1>, K2Smem::kThreads, K2Smem::kBytes);
  add("backproject_sr<table>", (const void*)backproject_sr_kernel<false, 1>, K2Smem::kThreads, K2Smem::kBytes);
  add("backproject_sr<table, pairs>", (const void*)backproject_sr_kernel<false, 2>, K2Smem::kThreads, K2PairSmem::kBytes);
  return QG_OK;
}

}  // namespace qg
