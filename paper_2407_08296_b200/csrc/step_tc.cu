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
// Warp roles: one TMA producer thread, one MMA issuer thread, (first kernel only) one loader thread
// for the M/V chunks, and four epilogue warps that read the accumulator with tcgen05.ld.  The
// accumulator is double buffered in tensor memory, so the epilogue of a tile overlaps the main
// loop of the next one.  Everything global the epilogue touches goes through shared memory in the
// 128-byte TMA swizzle: a thread reads/writes its own row with 16-byte accesses without bank
// conflicts, and global traffic stays fully coalesced.
//
// Every barrier wait is bounded; on expiry the kernel raises QG_DEV_WAIT_EXPIRED in the status word,
// stops taking tiles, releases its tensor memory and returns.
#include <cstring>

#include "sm100_ptx.cuh"
#include "step_epilogue.cuh"

namespace qg {

namespace {

using namespace ptx;

constexpr int kBK = 64;                 // K extent of one pipeline stage (elements)
constexpr int kBoxBytes = 64 * kBK * 2; // one TMA box of an operand: 64 x kBK bf16 = 8 KB
constexpr int kTileM = 128;             // accumulator rows (TMEM lanes)
constexpr int kChunk = 32;              // accumulator columns per tcgen05.ld

// One matrix of the step, as the kernels see it.  Tensor maps (row-major tensors, inner extent first):
//   mapP    P~  bf16 [m][r]       box 64 x 64, swizzle 128   A operand of both kernels
//   mapG    G   bf16 [m][ldg]     box 64 x 64, swizzle 128   B operand of the projection
//   mapN    N_b bf16 [r][ldn]     box 64 x 64, swizzle 128   B operand of the back-projection
//   mapNst  N_b bf16 [r][ldn]     box 32 x 128, swizzle 64   store from the Adam epilogue
//   mapM/V  fp32 [r][ldmv]        box 32 x 128, swizzle 128  load of the Adam epilogue
//   mapW    int8 [m][ldw]         box 128 x 128, swizzle 128 load of the requantizing epilogue
//   mapMst/Vst/Wst                the same tensors for the stores, with the inner extent rounded DOWN to
//                                 16 bytes: a TMA store clips at 16-byte granularity, so it would spill into
//                                 the row padding of a ragged matrix; the few tail columns are written with
//                                 plain stores instead (n_tma_mv / n_tma_w = columns the TMA stores cover).
struct alignas(64) TcProblem {
  CUtensorMap mapP, mapG, mapN, mapNst, mapM, mapV, mapW, mapMst, mapVst, mapWst;
  StepScalars sc;
  float* w_scales;
  float* w_zeros;
  float* dbgR;
  float* dbgN;
  float* dbgW;
  float* M;
  float* V;
  int8_t* w_codes;
  int64_t ldmv, ldw;
  int32_t m, n, r, ngroups, n_tma_mv, n_tma_w;
  int32_t k1_rblocks, k1_tiles, k1_tile0;
  int32_t k2_mblocks, k2_tiles, k2_tile0;
};
static_assert(sizeof(TcProblem) <= 2048, "TcProblem must fit the kernel parameter space");

__device__ __forceinline__ void raise_wait_expired(int32_t* status) {
  if (status) atomicOr(status, QG_DEV_WAIT_EXPIRED);
}

// ============================================================================================
// Kernel 1: projection + Adam
// ============================================================================================
template <int BN>
struct K1Smem {
  static constexpr int kStages = 3;
  static constexpr int kABytes = 2 * kBoxBytes;            // 128 (r) x 64 (m) bf16
  static constexpr int kBBytes = (BN / 64) * kBoxBytes;    // BN (n) x 64 (m) bf16
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kMvBufs = 3;
  static constexpr int kMBytes = kTileM * kChunk * 4;      // 16 KB
  static constexpr int kNBytes = kTileM * kChunk * 2;      // 8 KB
  static constexpr int kMvBufBytes = 2 * kMBytes + kNBytes;
  static constexpr int kBarOffset = kStages * kStageBytes + kMvBufs * kMvBufBytes;
  static constexpr int kBytes = kBarOffset + 256 + 1024;   // barriers + slack for 1024-byte alignment
};

template <int BN, bool SINGLE>
__global__ void __launch_bounds__(224, 1)
project_adam_kernel(const __grid_constant__ TcProblem single, const TcProblem* __restrict__ table, int nprob,
                    int total_tiles, int32_t* __restrict__ status) {
  using S = K1Smem<BN>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stage_base = smem;
  uint8_t* mv_base = smem + S::kStages * S::kStageBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::kBarOffset);
  uint64_t* full = bars;                         // [kStages]
  uint64_t* empty = bars + S::kStages;           // [kStages]
  uint64_t* acc_full = bars + 2 * S::kStages;    // [2]
  uint64_t* acc_empty = acc_full + 2;            // [2]
  uint64_t* mv_full = acc_empty + 2;             // [kMvBufs]
  uint64_t* mv_empty = mv_full + S::kMvBufs;     // [kMvBufs]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(mv_empty + S::kMvBufs);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const TcProblem* probs = SINGLE ? &single : table;

  if (threadIdx.x == 0) {
    for (int i = 0; i < S::kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 4); }
    for (int i = 0; i < S::kMvBufs; ++i) { mbar_init(&mv_full[i], 1); mbar_init(&mv_empty[i], 1); }
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // tile -> (problem, r block, n block); consecutive tiles share the n block, so that the G tile
  // one of them brings from HBM serves the others from L2
  auto locate = [&](int tile, int& pi) -> const TcProblem* {
    if (SINGLE) return probs;
    while (pi + 1 < nprob && tile >= probs[pi].k1_tile0 + probs[pi].k1_tiles) ++pi;
    return probs + pi;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int pi = 0;
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        const TcProblem* p = locate(tile, pi);
        const int local = tile - p->k1_tile0;
        const int r0 = (local % p->k1_rblocks) * kTileM, n0 = (local / p->k1_rblocks) * BN;
        const int kblocks = (p->m + kBK - 1) / kBK;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          const uint32_t ph = (it / S::kStages) & 1;
          if (!mbar_wait(&empty[s], ph ^ 1)) { ok = false; break; }
          uint8_t* sA = stage_base + s * S::kStageBytes;
          uint8_t* sB = sA + S::kABytes;
          mbar_arrive_expect_tx(&full[s], S::kStageBytes);
#pragma unroll
          for (int h = 0; h < 2; ++h) tma_load_2d(sA + h * kBoxBytes, &p->mapP, &full[s], r0 + 64 * h, kb * kBK);
#pragma unroll
          for (int h = 0; h < BN / 64; ++h) tma_load_2d(sB + h * kBoxBytes, &p->mapG, &full[s], n0 + 64 * h, kb * kBK);
        }
      }
      if (!ok) raise_wait_expired(status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kTileM, BN, true, true);
      int pi = 0;
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++tcount) {
        const TcProblem* p = locate(tile, pi);
        const int kblocks = (p->m + kBK - 1) / kBK;
        const uint32_t ab = tcount & 1;
        if (!mbar_wait(&acc_empty[ab], ((tcount >> 1) & 1) ^ 1)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + ab * BN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          if (!mbar_wait(&full[s], (it / S::kStages) & 1)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t aA = smem_u32(stage_base + s * S::kStageBytes);
          const uint32_t aB = aA + S::kABytes;
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            // both operands are MN-major: 16 K indices = two 8-index groups of 1024 bytes each
            const uint64_t da = umma_smem_desc_sw128(aA + k * 2048, kBoxBytes, 1024);
            const uint64_t db = umma_smem_desc_sw128(aB + k * 2048, kBoxBytes, 1024);
            umma_bf16(d_tmem, da, db, idesc, (kb | k) != 0);
          }
          umma_commit(&empty[s]);
        }
        if (ok) umma_commit(&acc_full[ab]);
      }
      if (!ok) raise_wait_expired(status);
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ loader of the M, V chunks
    if (lane == 0) {
      int pi = 0;
      uint32_t cc = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        const TcProblem* p = locate(tile, pi);
        const int local = tile - p->k1_tile0;
        const int r0 = (local % p->k1_rblocks) * kTileM, n0 = (local / p->k1_rblocks) * BN;
        const int nchunks = min(BN / kChunk, (p->n - n0 + kChunk - 1) / kChunk);
        for (int c = 0; c < nchunks; ++c, ++cc) {
          const int b = cc % S::kMvBufs;
          if (!mbar_wait(&mv_empty[b], ((cc / S::kMvBufs) & 1) ^ 1)) { ok = false; break; }
          uint8_t* buf = mv_base + b * S::kMvBufBytes;
          mbar_arrive_expect_tx(&mv_full[b], 2 * S::kMBytes);
          tma_load_2d(buf, &p->mapM, &mv_full[b], n0 + c * kChunk, r0);
          tma_load_2d(buf + S::kMBytes, &p->mapV, &mv_full[b], n0 + c * kChunk, r0);
        }
      }
      if (!ok) raise_wait_expired(status);
    }
  } else {
    // ------------------------------------------------------------------ epilogue: Adam on the tile
    const int q = warp & 3;                         // TMEM lane quarter this warp may access
    const int row = q * 32 + lane;                  // accumulator row = row of the r block
    const bool elected = (threadIdx.x == 96);       // first epilogue thread issues the TMA stores
    int pi = 0;
    uint32_t cc = 0, tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++tcount) {
      const TcProblem* p = locate(tile, pi);
      const int local = tile - p->k1_tile0;
      const int r0 = (local % p->k1_rblocks) * kTileM, n0 = (local / p->k1_rblocks) * BN;
      const int nchunks = min(BN / kChunk, (p->n - n0 + kChunk - 1) / kChunk);
      const StepScalars sc = p->sc;
      const float inv_b1 = 1.0f / sc.bias1, inv_b2 = 1.0f / sc.bias2;
      const uint32_t ab = tcount & 1;
      ok = named_bar_and(1, 128, mbar_wait(&acc_full[ab], (tcount >> 1) & 1));
      if (!ok) break;
      tc_fence_after_sync();
      for (int c = 0; c < nchunks; ++c, ++cc) {
        const int b = cc % S::kMvBufs;
        ok = named_bar_and(1, 128, mbar_wait(&mv_full[b], (cc / S::kMvBufs) & 1));
        if (!ok) break;
        uint32_t acc[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + ab * BN + c * kChunk, acc);
        tmem_ld_wait();
        uint8_t* buf = mv_base + b * S::kMvBufBytes;
        float4* Mrow = reinterpret_cast<float4*>(buf + row * 128);
        float4* Vrow = reinterpret_cast<float4*>(buf + S::kMBytes + row * 128);
        uint2* Nrow = reinterpret_cast<uint2*>(buf + 2 * S::kMBytes + row * 64);
        const bool tap = (p->dbgR != nullptr || p->dbgN != nullptr) && (r0 + row < p->r);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int pj = j ^ (row & 7);             // 128-byte swizzle: 16-byte chunk j lives at j ^ (row % 8)
          float4 m4 = Mrow[pj], v4 = Vrow[pj];
          float mm[4] = {m4.x, m4.y, m4.z, m4.w}, vv[4] = {v4.x, v4.y, v4.z, v4.w}, nn[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float rr = __uint_as_float(acc[4 * j + e]);
            mm[e] = fmaf(sc.beta1, mm[e], sc.one_minus_beta1 * rr);
            vv[e] = fmaf(sc.beta2, vv[e], sc.one_minus_beta2 * rr * rr);
            nn[e] = __fdividef(mm[e] * inv_b1, sqrtf(vv[e] * inv_b2) + sc.eps);
          }
          Mrow[pj] = make_float4(mm[0], mm[1], mm[2], mm[3]);
          Vrow[pj] = make_float4(vv[0], vv[1], vv[2], vv[3]);
          if (n0 + c * kChunk + 4 * j == p->n_tma_mv && r0 + row < p->r) {   // ragged tail: at most 3 columns
#pragma unroll
            for (int e = 0; e < 3; ++e) {
              if (e < p->n - p->n_tma_mv) {
                p->M[(int64_t)(r0 + row) * p->ldmv + p->n_tma_mv + e] = mm[e];
                p->V[(int64_t)(r0 + row) * p->ldmv + p->n_tma_mv + e] = vv[e];
              }
            }
          }
          uint2 nb;
          nb.x = (uint32_t)float_to_bf16_bits(nn[0]) | ((uint32_t)float_to_bf16_bits(nn[1]) << 16);
          nb.y = (uint32_t)float_to_bf16_bits(nn[2]) | ((uint32_t)float_to_bf16_bits(nn[3]) << 16);
          // 64-byte swizzle of the bf16 tile: 16-byte chunk (j / 2) lives at (j / 2) ^ ((row / 2) % 4)
          Nrow[(((j >> 1) ^ ((row >> 1) & 3)) << 1) | (j & 1)] = nb;
          if (tap) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int col = n0 + c * kChunk + 4 * j + e;
              if (col < p->n) {
                if (p->dbgR) p->dbgR[(int64_t)(r0 + row) * p->ldmv + col] = __uint_as_float(acc[4 * j + e]);
                if (p->dbgN) p->dbgN[(int64_t)(r0 + row) * p->ldmv + col] = nn[e];
              }
            }
          }
        }
        fence_proxy_async_smem();
        named_bar_sync(1, 128);
        if (elected) {
          if (n0 + c * kChunk < p->n_tma_mv) {
            tma_store_2d(&p->mapMst, buf, n0 + c * kChunk, r0);
            tma_store_2d(&p->mapVst, buf + S::kMBytes, n0 + c * kChunk, r0);
          }
          tma_store_2d(&p->mapNst, buf + 2 * S::kMBytes, n0 + c * kChunk, r0);
          tma_commit_group();
          if (cc >= 1) {                             // the previous chunk's buffer has been read out
            tma_wait_group_read<1>();
            mbar_arrive(&mv_empty[(cc - 1) % S::kMvBufs]);
          }
        }
      }
      if (!ok) break;
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[ab]);
    }
    if (elected) tma_wait_group<0>();
    if (!ok && lane == 0) raise_wait_expired(status);
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 2 * BN);
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
  static constexpr int kBytes = kBarOffset + 256 + 1024;
};

// Pre-rounding weight of one element: W' = W^ - lr*alpha*D - lr*wd*W^ with W^ = (q - z) * s.
__device__ __forceinline__ float weight_pre(float qf, float z, float s, float d, const StepScalars& sc) {
  const float wh = __fmul_rn(__fsub_rn(qf, z), s);
  return fmaf(-sc.lr_alpha, d, fmaf(-sc.lr_wd, wh, wh));
}

template <bool SINGLE>
__global__ void __launch_bounds__(192, 1)
backproject_sr_kernel(const __grid_constant__ TcProblem single, const TcProblem* __restrict__ table, int nprob,
                      int total_tiles, int32_t* __restrict__ status) {
  using S = K2Smem;
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

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const TcProblem* probs = SINGLE ? &single : table;

  if (threadIdx.x == 0) {
    for (int i = 0; i < S::kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 4); }
    for (int i = 0; i < S::kCodeBufs; ++i) { mbar_init(&code_full[i], 1); mbar_init(&code_empty[i], 1); }
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // tile -> (problem, m block, n block); consecutive tiles share the n block of N_b
  auto locate = [&](int tile, int& pi) -> const TcProblem* {
    if (SINGLE) return probs;
    while (pi + 1 < nprob && tile >= probs[pi].k2_tile0 + probs[pi].k2_tiles) ++pi;
    return probs + pi;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int pi = 0;
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++tcount) {
        const TcProblem* p = locate(tile, pi);
        const int local = tile - p->k2_tile0;
        const int m0 = (local % p->k2_mblocks) * kTileM, n0 = (local / p->k2_mblocks) * S::kBN;
        const int cb = tcount % S::kCodeBufs;
        if (!mbar_wait(&code_empty[cb], ((tcount / S::kCodeBufs) & 1) ^ 1)) { ok = false; break; }
        uint8_t* cbuf = code_base + cb * S::kCodeBytes;
        mbar_arrive_expect_tx(&code_full[cb], S::kCodeBytes);
        tma_load_2d(cbuf, &p->mapW, &code_full[cb], n0, m0);
        tma_load_2d(cbuf + S::kCodeBytes / 2, &p->mapW, &code_full[cb], n0 + 128, m0);
        const int kblocks = (p->r + kBK - 1) / kBK;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          if (!mbar_wait(&empty[s], ((it / S::kStages) & 1) ^ 1)) { ok = false; break; }
          uint8_t* sA = stage_base + s * S::kStageBytes;
          uint8_t* sB = sA + S::kABytes;
          mbar_arrive_expect_tx(&full[s], S::kStageBytes);
#pragma unroll
          for (int h = 0; h < 2; ++h) tma_load_2d(sA + h * kBoxBytes, &p->mapP, &full[s], kb * kBK, m0 + 64 * h);
#pragma unroll
          for (int h = 0; h < 4; ++h) tma_load_2d(sB + h * kBoxBytes, &p->mapN, &full[s], n0 + 64 * h, kb * kBK);
        }
      }
      if (!ok) raise_wait_expired(status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kTileM, S::kBN, false, true);
      int pi = 0;
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++tcount) {
        const TcProblem* p = locate(tile, pi);
        const int kblocks = (p->r + kBK - 1) / kBK;
        const uint32_t ab = tcount & 1;
        if (!mbar_wait(&acc_empty[ab], ((tcount >> 1) & 1) ^ 1)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + ab * S::kBN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          if (!mbar_wait(&full[s], (it / S::kStages) & 1)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t aA = smem_u32(stage_base + s * S::kStageBytes);
          const uint32_t aB = aA + S::kABytes;
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            // A is K-major (rows of 128 bytes, 16 K indices = 32 bytes further along the row),
            // B is MN-major (16 K indices = two 8-index groups of 1024 bytes)
            const uint64_t da = umma_smem_desc_sw128(aA + k * 32, 16, 1024);
            const uint64_t db = umma_smem_desc_sw128(aB + k * 2048, kBoxBytes, 1024);
            umma_bf16(d_tmem, da, db, idesc, (kb | k) != 0);
          }
          umma_commit(&empty[s]);
        }
        if (ok) umma_commit(&acc_full[ab]);
      }
      if (!ok) raise_wait_expired(status);
    }
  } else {
    // ------------------------------------------------------------------ epilogue: one thread = one row = one group
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const bool elected = (threadIdx.x == 64);
    int pi = 0;
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++tcount) {
      const TcProblem* p = locate(tile, pi);
      const int local = tile - p->k2_tile0;
      const int m0 = (local % p->k2_mblocks) * kTileM, nblk = local / p->k2_mblocks, n0 = nblk * S::kBN;
      const int gi = m0 + row;                       // global row
      const bool row_ok = gi < p->m;
      const int ncols = min(S::kBN, p->n - n0);      // valid columns of this (possibly ragged) group
      const StepScalars sc = p->sc;
      float s_old = 1.f, z_old = 0.f;
      if (row_ok) {
        s_old = __ldg(p->w_scales + (int64_t)gi * p->ngroups + nblk);
        z_old = __ldg(p->w_zeros + (int64_t)gi * p->ngroups + nblk);
      }
      const uint32_t ab = tcount & 1;
      const int cb = tcount % S::kCodeBufs;
      ok = mbar_wait(&code_full[cb], (tcount / S::kCodeBufs) & 1) && mbar_wait(&acc_full[ab], (tcount >> 1) & 1);
      ok = named_bar_and(1, 128, ok);
      if (!ok) break;
      tc_fence_after_sync();
      uint8_t* cbuf = code_base + cb * S::kCodeBytes;
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + ab * S::kBN;
      // codes of column 16*k16 .. +15 of this row: box (k16 / 8), 16-byte chunk (k16 % 8) ^ (row % 8)
      auto code_ptr = [&](int k16) -> uint4* {
        return reinterpret_cast<uint4*>(cbuf + (k16 >> 3) * (S::kCodeBytes / 2) + row * 128 + (((k16 & 7) ^ (row & 7)) << 4));
      };

      // ---- pass 1: group minimum and maximum of W'
      float mn = INFINITY, mx = -INFINITY;
      for (int c = 0; c < S::kBN / kChunk; ++c) {
        uint32_t acc[32];
        tmem_ld_32x32(tacc + c * kChunk, acc);
        tmem_ld_wait();
#pragma unroll
        for (int hlf = 0; hlf < 2; ++hlf) {
          const uint4 cw = *code_ptr(2 * c + hlf);
          const uint32_t w4[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float qf = (float)(int8_t)((w4[e >> 2] >> (8 * (e & 3))) & 0xFFu);
            const float w = weight_pre(qf, z_old, s_old, __uint_as_float(acc[16 * hlf + e]), sc);
            if (c * kChunk + 16 * hlf + e < ncols) { mn = fminf(mn, w); mx = fmaxf(mx, w); }
          }
        }
      }
      const GroupParams gp = group_params<8>(mn, mx);
      if (row_ok) {
        p->w_scales[(int64_t)gi * p->ngroups + nblk] = gp.s;
        p->w_zeros[(int64_t)gi * p->ngroups + nblk] = gp.z;
      }

      // ---- pass 2: stochastic rounding to the new grid, codes written back in place
      for (int c = 0; c < S::kBN / kChunk; ++c) {
        uint32_t acc[32];
        tmem_ld_32x32(tacc + c * kChunk, acc);
        tmem_ld_wait();
#pragma unroll
        for (int hlf = 0; hlf < 2; ++hlf) {
          uint4* cp = code_ptr(2 * c + hlf);
          const uint4 cw = *cp;
          const uint32_t w4[4] = {cw.x, cw.y, cw.z, cw.w};
          uint32_t o4[4] = {0, 0, 0, 0};
#pragma unroll
          for (int e8 = 0; e8 < 2; ++e8) {
            float h[8];
            sr_lanes8(sc, (uint32_t)gi, (uint32_t)((n0 + c * kChunk + 16 * hlf + 8 * e8) >> 3), h);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int ee = 8 * e8 + e;
              const float qf = (float)(int8_t)((w4[ee >> 2] >> (8 * (ee & 3))) & 0xFFu);
              const float w = weight_pre(qf, z_old, s_old, __uint_as_float(acc[16 * hlf + ee]), sc);
              const int code = (int)sr_code(w, gp, h[e]);
              o4[ee >> 2] |= (uint32_t)(code & 0xFF) << (8 * (ee & 3));
              if (p->dbgW && row_ok && (n0 + c * kChunk + 16 * hlf + ee) < p->n)
                p->dbgW[(int64_t)gi * p->ldw + n0 + c * kChunk + 16 * hlf + ee] = w;
            }
          }
          *cp = make_uint4(o4[0], o4[1], o4[2], o4[3]);
          if (n0 + c * kChunk + 16 * hlf == p->n_tma_w && row_ok) {          // ragged tail: at most 15 columns
            int8_t* out = p->w_codes + (int64_t)gi * p->ldw + p->n_tma_w;
#pragma unroll
            for (int e = 0; e < 15; ++e)
              if (e < p->n - p->n_tma_w) out[e] = (int8_t)((o4[e >> 2] >> (8 * (e & 3))) & 0xFFu);
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[ab]);

      // ---- coalesced write-back of the tile's codes
      fence_proxy_async_smem();
      named_bar_sync(1, 128);
      if (elected) {
        if (n0 < p->n_tma_w) tma_store_2d(&p->mapWst, cbuf, n0, m0);
        if (n0 + 128 < p->n_tma_w) tma_store_2d(&p->mapWst, cbuf + S::kCodeBytes / 2, n0 + 128, m0);
        tma_commit_group();
        tma_wait_group_read<0>();
        mbar_arrive(&code_empty[cb]);
      }
    }
    if (elected) tma_wait_group<0>();
    if (!ok && lane == 0) raise_wait_expired(status);
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

// ============================================================================================
// host side
// ============================================================================================
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      p = nullptr;
    (void)cudaGetLastError();
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Row-major 2-D tensor [outer][pitch], `inner` valid elements per row; out-of-range elements read as zero
// and are not written.
bool make_map(CUtensorMap* map, CUtensorMapDataType dt, int elem_bytes, const void* base, int64_t inner, int64_t outer,
              int64_t pitch_elems, int box_inner, int box_outer, CUtensorMapSwizzle sw) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t gdim[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  const cuuint64_t gstr[1] = {(cuuint64_t)pitch_elems * elem_bytes};
  const cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, dt, 2, const_cast<void*>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct TcWorkspace {
  uint16_t* Pt;
  uint16_t* Nb;
  int64_t ldn;
};

TcWorkspace carve(const StepArgs& a) {
  TcWorkspace w;
  w.Pt = reinterpret_cast<uint16_t*>(a.ws);
  w.Nb = reinterpret_cast<uint16_t*>(reinterpret_cast<char*>(a.ws) + round_up(a.m * a.r * 2, 1024));
  w.ldn = round_up(a.n, 64);
  return w;
}

int fill_problem(const StepArgs& a, TcProblem* p, int bn) {
  memset(p, 0, sizeof(*p));
  const TcWorkspace w = carve(a);
  bool ok = true;
  ok &= make_map(&p->mapP, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, w.Pt, a.r, a.m, a.r, 64, kBK, CU_TENSOR_MAP_SWIZZLE_128B);
  ok &= make_map(&p->mapG, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.G, a.n, a.m, a.ldg, 64, kBK, CU_TENSOR_MAP_SWIZZLE_128B);
  ok &= make_map(&p->mapN, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, w.Nb, a.n, a.r, w.ldn, 64, kBK, CU_TENSOR_MAP_SWIZZLE_128B);
  ok &= make_map(&p->mapNst, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, w.Nb, a.n, a.r, w.ldn, kChunk, kTileM,
                 CU_TENSOR_MAP_SWIZZLE_64B);
  ok &= make_map(&p->mapM, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.M, a.n, a.r, a.ldmv, kChunk, kTileM,
                 CU_TENSOR_MAP_SWIZZLE_128B);
  ok &= make_map(&p->mapV, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.V, a.n, a.r, a.ldmv, kChunk, kTileM,
                 CU_TENSOR_MAP_SWIZZLE_128B);
  ok &= make_map(&p->mapW, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.W.codes, a.n, a.m, a.W.ld, 128, kTileM,
                 CU_TENSOR_MAP_SWIZZLE_128B);
  const int64_t n4 = a.n & ~int64_t(3), n16 = a.n & ~int64_t(15);
  ok &= make_map(&p->mapMst, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.M, n4 > 0 ? n4 : 4, a.r, a.ldmv, kChunk, kTileM,
                 CU_TENSOR_MAP_SWIZZLE_128B);
  ok &= make_map(&p->mapVst, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.V, n4 > 0 ? n4 : 4, a.r, a.ldmv, kChunk, kTileM,
                 CU_TENSOR_MAP_SWIZZLE_128B);
  ok &= make_map(&p->mapWst, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.W.codes, n16 > 0 ? n16 : 16, a.m, a.W.ld, 128, kTileM,
                 CU_TENSOR_MAP_SWIZZLE_128B);
  p->n_tma_mv = (int32_t)n4;
  p->n_tma_w = (int32_t)n16;
  p->M = a.M; p->V = a.V; p->w_codes = reinterpret_cast<int8_t*>(a.W.codes);
  if (!ok) {
    note_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled");
    return QG_CUDA_ERROR;
  }
  p->sc = a.sc;
  p->w_scales = a.W.scales;
  p->w_zeros = a.W.zeros;
  p->dbgR = a.dbg.R; p->dbgN = a.dbg.N; p->dbgW = a.dbg.W_pre;
  p->ldmv = a.ldmv; p->ldw = a.W.ld;
  p->m = (int32_t)a.m; p->n = (int32_t)a.n; p->r = (int32_t)a.r;
  p->ngroups = (int32_t)ceil_div(a.n, kGroup);
  p->k1_rblocks = (int32_t)ceil_div(a.r, kTileM);
  p->k1_tiles = p->k1_rblocks * (int32_t)ceil_div(a.n, bn);
  p->k2_mblocks = (int32_t)ceil_div(a.m, kTileM);
  p->k2_tiles = p->k2_mblocks * (int32_t)ceil_div(a.n, K2Smem::kBN);
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

template <class K>
int set_smem(K kernel, int bytes) {
  QG_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  return QG_OK;
}

}  // namespace

size_t tc_workspace_bytes(int64_t m, int64_t n, int64_t r) {
  return (size_t)round_up(m * r * 2, 1024) + (size_t)round_up(r * round_up(n, 64) * 2, 1024);
}

int launch_project_step_tc(const StepArgs& a, cudaStream_t st) {
  const TcWorkspace w = carve(a);
  int rc = launch_dequant_p(a.P, w.Pt, a.r, st);
  if (rc != QG_OK) return rc;
  TcProblem prob;
  constexpr int BN = 128;
  rc = fill_problem(a, &prob, BN);
  if (rc != QG_OK) return rc;
  const int sms = sm_count();
  {
    auto kern = project_adam_kernel<BN, true>;
    rc = set_smem(kern, K1Smem<BN>::kBytes);
    if (rc != QG_OK) return rc;
    const int grid = prob.k1_tiles < sms ? prob.k1_tiles : sms;
    kern<<<grid, 224, K1Smem<BN>::kBytes, st>>>(prob, nullptr, 1, prob.k1_tiles, a.status);
    QG_LAUNCH_CHECK();
  }
  {
    auto kern = backproject_sr_kernel<true>;
    rc = set_smem(kern, K2Smem::kBytes);
    if (rc != QG_OK) return rc;
    const int grid = prob.k2_tiles < sms ? prob.k2_tiles : sms;
    kern<<<grid, 192, K2Smem::kBytes, st>>>(prob, nullptr, 1, prob.k2_tiles, a.status);
    QG_LAUNCH_CHECK();
  }
  return QG_OK;
}

}  // namespace qg
