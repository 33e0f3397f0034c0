// The INT8 linear layer of App. A as tcgen05 GEMMs that take the INT8 weight as it is stored:
//
//   forward          Y^T = W~ X^T       (m x T)    A = W~  from tensor memory, B = X K-major    (K = n)
//   input gradient   dX  = dY W~        (T x n)    A = dY  K-major,   B = W~    MN-major        (K = m)
//   weight gradient  G   = dY^T X       (m x n)    A = dY^T MN-major, B = X     MN-major        (K = T)
//
// with W~ = bf16((q - z) * s), the weight dequantized in binary32 per group of 256 (Sec. 3.1) and rounded once
// to the activations' type.  W~ never exists in global memory: the INT8 codes of a tile arrive in shared memory
// by TMA and converter warps dequantize them straight into the operand the MMA reads - tensor memory for the
// forward product (second kernel below), the 128-byte-swizzled shared-memory layout for the input gradient.
// The accumulator (fp32, tensor memory) leaves as bfloat16.  The weight gradient has no quantized operand: both
// tiles come by TMA in MN-major form, and its output is the matrix G the optimizer step reads.
//
// One persistent CTA per SM, tiles of 128 x 256.  The first kernel (input and weight gradient) keeps two
// accumulators in tensor memory so that the epilogue of a tile overlaps the main loop of the next; warp roles:
// 0 TMA producer (A, and B of the weight gradient), 1 MMA issuer and tensor-memory owner, 2 TMA producer of the
// INT8 tiles, 4-7 epilogue, 8-15 converters.
// Every barrier wait is bounded; a wait that runs out raises QG_DEV_WAIT_EXPIRED and the role stops.
#include <cstring>

#include "qg_common.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace qg {

using namespace ptx;

namespace {

constexpr int kBK = 64;        // K extent of a pipeline stage
constexpr int kTileM = 128;    // accumulator rows (TMEM lanes)
constexpr int kTileN = 256;    // accumulator columns; a multiple of the quantization group along n
constexpr int kSlab = 64 * kBK * 2;   // one 64-wide MN-major slab of a stage: 64 K rows of 128 bytes

enum : int { kForward = 0, kInputGrad = 1, kWeightGrad = 2 };

struct LinArgs {
  CUtensorMap mapA;            // bf16 activations: K-major 2-D (X of the forward product, where it is the MMA's B
                               // operand; dY of the input gradient) or chunked 3-D (dY of the weight gradient)
  CUtensorMap mapB;            // INT8 codes of W (2-D, bytes) or, for the weight gradient, X chunked 3-D
  const float* scales;         // of W: [w_rows][ngroups]
  const float* zeros;
  int32_t ngroups, w_rows;
  uint16_t* D;                 // bf16 output, row-major
  int64_t ldd;
  int32_t rows, cols, K;       // accumulator extents (forward: rows of W x rows of X) and contraction length
  int32_t mblocks, nblocks;
};

template <int MODE>
struct LinSmem {
  static constexpr bool kConvert = MODE != kWeightGrad;
  // The input gradient takes TWO row blocks of dY per tile of W: a converted B tile then serves two MMAs, which
  // halves, per flop, the shared-memory traffic of the conversion (codes in, codes read, bf16 written) that bounds
  // this product.  Both accumulators together fill tensor memory, so its epilogue does not overlap the next main loop.
  static constexpr int kMT = MODE == kInputGrad ? 2 : 1;
  static constexpr int kABytes = kMT * kTileM * kBK * 2;       // 16 KB per row block
  static constexpr int kBBytes = kTileN * kBK * 2;             // 32 KB
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = kConvert ? 2 : 4;
  static constexpr int kRawBytes = kTileN * kBK;               // one INT8 tile: 16 KB
  static constexpr int kRawStages = kConvert ? 3 : 0;
  static constexpr int kBarOffset = kStages * kStageBytes + kRawStages * kRawBytes;
  static constexpr int kBytes = kBarOffset + 256 + 1024;       // barriers + slack for 1024-byte alignment
  static constexpr int kEpiWarps = 4, kConvWarps = 8;
  static constexpr int kThreads = (4 + kEpiWarps + kConvWarps) * 32;
  static_assert(kBytes <= 227 * 1024, "shared memory budget");
};

__device__ __forceinline__ void raise_expired(int32_t* status) {
  if (status) atomicOr(status, QG_DEV_WAIT_EXPIRED);
}

// Sixteen INT8 codes (one 16-byte word) -> sixteen bfloat16 of (q - z) * s, as two 16-byte words.
// bias = 2^23 + 128 + z: the code byte with its sign bit flipped is q + 128, placed in the low mantissa
// byte of 2^23 it reads as the float 2^23 + 128 + q, and subtracting bias leaves q - z exactly; one
// binary32 multiplication and one rounding to bfloat16 follow, the same two roundings as the definition.
__device__ __forceinline__ void dequant16(const uint4 codes, float bias, float s, uint4& lo, uint4& hi) {
  const uint32_t w[4] = {codes.x ^ 0x80808080u, codes.y ^ 0x80808080u, codes.z ^ 0x80808080u, codes.w ^ 0x80808080u};
  const float2 nb = make_float2(-bias, -bias), s2 = make_float2(s, s);
  uint32_t out[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 a = make_float2(__uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7440)),
                                 __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7441)));
    const float2 b = make_float2(__uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7442)),
                                 __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7443)));
    const float2 va = mul2(add2(a, nb), s2), vb = mul2(add2(b, nb), s2);
    __nv_bfloat162 pa = __floats2bfloat162_rn(va.x, va.y), pb = __floats2bfloat162_rn(vb.x, vb.y);
    out[2 * i] = *reinterpret_cast<uint32_t*>(&pa);
    out[2 * i + 1] = *reinterpret_cast<uint32_t*>(&pb);
  }
  lo = make_uint4(out[0], out[1], out[2], out[3]);
  hi = make_uint4(out[4], out[5], out[6], out[7]);
}

template <int MODE>
__global__ void __launch_bounds__(LinSmem<MODE>::kThreads, 1)
int8_linear_kernel(const __grid_constant__ LinArgs a, int32_t* __restrict__ status) {
  using S = LinSmem<MODE>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stage_base = smem;
  uint8_t* raw_base = smem + S::kStages * S::kStageBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::kBarOffset);
  uint64_t* full = bars;
  uint64_t* empty = full + S::kStages;
  uint64_t* raw_full = empty + S::kStages;
  uint64_t* raw_empty = raw_full + 4;
  uint64_t* acc_full = raw_empty + 4;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < S::kStages; ++i) {
      mbar_init(&full[i], S::kConvert ? 1 + S::kConvWarps / 2 : 1);   // the TMA producer, and the converter warps of one group
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < S::kRawStages; ++i) { mbar_init(&raw_full[i], 1); mbar_init(&raw_empty[i], S::kConvWarps / 2); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], S::kEpiWarps); }
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // tile t -> (m block, n block): consecutive tiles (concurrent CTAs) share the n block, i.e. the same
  // columns of B, which for two of the three products is the weight
  const int total = a.mblocks * a.nblocks;
  const int kblocks = (a.K + kBK - 1) / kBK;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer of A (and bf16 B)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < total; t += gridDim.x) {
        const int m0 = (t % a.mblocks) * (S::kMT * kTileM), n0 = (t / a.mblocks) * kTileN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          if (!mbar_wait(&empty[s], ((it / S::kStages) & 1) ^ 1)) { ok = false; break; }
          uint8_t* sA = stage_base + s * S::kStageBytes;
          if (MODE == kWeightGrad) {
            mbar_arrive_expect_tx(&full[s], S::kStageBytes);
            tma_load_3d(sA, &a.mapA, &full[s], 0, kb * kBK, m0 / 64);
            tma_load_3d(sA + S::kABytes, &a.mapB, &full[s], 0, kb * kBK, n0 / 64);
          } else {
            mbar_arrive_expect_tx(&full[s], S::kABytes);
#pragma unroll
            for (int h = 0; h < S::kMT; ++h)       // rows past the matrix read as zero
              tma_load_2d(sA + h * (S::kABytes / S::kMT), &a.mapA, &full[s], kb * kBK, m0 + h * kTileM);
          }
        }
      }
      if (!ok) raise_expired(status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kTileM, kTileN, MODE == kWeightGrad, true);
      // K-major: rows of 128 bytes, 8-row groups 1024 bytes apart, 16 K indices = 32 bytes along the row.
      // MN-major: 64-wide slabs of kSlab bytes, 8 K indices = 1024 bytes, 16 K indices = 2048 bytes.
      const uint64_t desc_a0 = MODE == kWeightGrad ? umma_smem_desc_sw128(smem_u32(stage_base), kSlab, 1024)
                                                   : umma_smem_desc_sw128(smem_u32(stage_base), 16, 1024);
      const uint64_t desc_b0 = umma_smem_desc_sw128(smem_u32(stage_base) + S::kABytes, kSlab, 1024);
      constexpr uint64_t astep = MODE == kWeightGrad ? (2048 >> 4) : (32 >> 4);
      constexpr uint64_t bstep = 2048 >> 4;
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < total; t += gridDim.x, ++tcount) {
        // one row block per tile: two accumulators of 256 columns take alternate tiles; two row blocks per tile: the
        // tile's two accumulators are the whole of tensor memory and barrier 0 alone paces the tiles
        const uint32_t ab = S::kMT == 1 ? (tcount & 1) : 0u;
        const uint32_t use = S::kMT == 1 ? (tcount >> 1) : tcount;
        if (!mbar_wait(&acc_empty[ab], (use & 1) ^ 1)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + ab * kTileN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          if (!mbar_wait(&full[s], (it / S::kStages) & 1)) { ok = false; break; }
          tc_fence_after_sync();
          const uint64_t da = desc_a0 + (uint64_t)((s * S::kStageBytes) >> 4);
          const uint64_t db = desc_b0 + (uint64_t)((s * S::kStageBytes) >> 4);
#pragma unroll
          for (int h = 0; h < S::kMT; ++h)
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)
              umma_bf16(d_tmem + h * kTileN, da + (uint64_t)((h * (S::kABytes / S::kMT)) >> 4) + k * astep, db + k * bstep, idesc,
                        (kb | k) != 0);
          umma_commit(&empty[s]);
        }
        if (ok) umma_commit(&acc_full[ab]);
      }
      if (!ok) raise_expired(status);
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ TMA producer of the INT8 tiles
    if (S::kConvert && lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < total; t += gridDim.x) {
        const int n0 = (t / a.mblocks) * kTileN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int rs = it % 3;
          if (!mbar_wait(&raw_empty[rs], ((it / 3) & 1) ^ 1)) { ok = false; break; }
          mbar_arrive_expect_tx(&raw_full[rs], S::kRawBytes);
          // 64 rows of W (the tile's K) x 256 bytes along n (its N), no swizzle
          tma_load_2d(raw_base + rs * S::kRawBytes, &a.mapB, &raw_full[rs], n0, kb * kBK);
        }
      }
      if (!ok) raise_expired(status);
    }
  } else if (warp >= 4 && warp < 4 + S::kEpiWarps) {
    // ------------------------------------------------------------------ epilogue: fp32 accumulator -> bf16
    const int q = warp & 3;
    uint32_t tcount = 0;
    bool ok = true;
    for (int t = blockIdx.x; ok && t < total; t += gridDim.x, ++tcount) {
      const int m0 = (t % a.mblocks) * (S::kMT * kTileM), n0 = (t / a.mblocks) * kTileN;
      const uint32_t ab = S::kMT == 1 ? (tcount & 1) : 0u;
      const uint32_t use = S::kMT == 1 ? (tcount >> 1) : tcount;
      if (!mbar_wait(&acc_full[ab], use & 1)) { ok = false; break; }
      tc_fence_after_sync();
#pragma unroll 1
      for (int cc = 0; cc < S::kMT * (kTileN / 32); ++cc) {
        const int h = cc / (kTileN / 32), c = cc % (kTileN / 32);      // row block of the tile, 32-column piece
        const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (ab + h) * kTileN;
        const int row = m0 + h * kTileM + q * 32 + lane;
        uint16_t* drow = a.D + (int64_t)row * a.ldd;
        uint32_t v[32];
        tmem_ld_32x32(tacc + 32 * c, v);
        tmem_ld_wait();
        if (cc == S::kMT * (kTileN / 32) - 1) {        // every read of this tile's accumulators has landed
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&acc_empty[ab]);
        }
        const int col = n0 + 32 * c;
        if (row < a.rows && col < a.cols) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
            pk[i] = *reinterpret_cast<uint32_t*>(&h);
          }
          if (col + 32 <= a.cols) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              *reinterpret_cast<uint4*>(drow + col + 8 * i) = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (col + i < a.cols) drow[col + i] = (uint16_t)((i & 1) ? (pk[i >> 1] >> 16) : (pk[i >> 1] & 0xFFFFu));
          }
        }
      }
    }
    if (!ok && lane == 0) raise_expired(status);
  } else if (S::kConvert && warp >= 8) {
    // ------------------------------------------------------------------ converters: INT8 tile -> bf16 operand
    // Two groups of four warps take alternate K blocks, so that the chain of one block (wait, load, convert,
    // store, fence, arrive) overlaps that of the next; a thread converts two rows of the tile.
    const int grp = (warp - 8) >> 2, lt = (threadIdx.x - 256) & 127;
    uint32_t it = 0;
    bool ok = true;
    for (int t = blockIdx.x; ok && t < total; t += gridDim.x) {
      const int n0 = (t / a.mblocks) * kTileN;
      for (int kb = 0; kb < kblocks; ++kb, ++it) {
        if ((int)(it & 1) != grp) continue;
        // rows 64 kb + lt / 4 and + 32 of W, scale of group n0 / 256
        float sc[2], bias[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int wr = kb * kBK + (lt >> 2) + 32 * h;
          const int64_t idx = (int64_t)wr * a.ngroups + n0 / kGroup;
          const bool valid = wr < a.w_rows;
          sc[h] = valid ? __ldg(a.scales + idx) : 0.f;
          bias[h] = 8388736.0f + (valid ? __ldg(a.zeros + idx) : 0.f);     // 2^23 + 128 + z
        }
        const int rs = it % 3, s = it % S::kStages;
        if (!mbar_wait(&raw_full[rs], (it / 3) & 1) || !mbar_wait(&empty[s], ((it / S::kStages) & 1) ^ 1)) { ok = false; break; }
        const uint8_t* raw = raw_base + rs * S::kRawBytes;
        uint8_t* sB = stage_base + s * S::kStageBytes + S::kABytes;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          // raw: [64 rows][256 bytes]; operand (MN-major): slab i holds columns 64 i .. 64 i + 63 as
          // [64 K rows][128 bytes], 16-byte piece j of row k stored at j ^ (k & 7)
          const int k = (lt >> 2) + 32 * h, q4 = lt & 3;
          const uint8_t* rrow = raw + k * 256 + q4 * 16;
          uint8_t* orow = sB + k * 128;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint4 codes = *reinterpret_cast<const uint4*>(rrow + i * 64);
            uint4 lo, hi;
            dequant16(codes, bias[h], sc[h], lo, hi);
            *reinterpret_cast<uint4*>(orow + i * kSlab + (((2 * q4) ^ (k & 7)) << 4)) = lo;
            *reinterpret_cast<uint4*>(orow + i * kSlab + (((2 * q4 + 1) ^ (k & 7)) << 4)) = hi;
          }
        }
        fence_proxy_async_smem();                      // the MMA reads these stores through the async proxy
        __syncwarp();
        if (lane == 0) { mbar_arrive(&full[s]); mbar_arrive(&raw_empty[rs]); }
      }
    }
    if (!ok && lane == 0) raise_expired(status);
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

// ----------------------------------------------------------------------------------------------------------
// The forward product with the converted weight handed to the MMA through TENSOR memory instead of shared
// memory.  The product is computed transposed, Y^T = W~ X^T: the accumulator's 128 rows are rows of W, its 256
// columns are rows of X (tokens); operand A is a 128 x 64 tile of W~ that a converter thread per row writes with
// one tcgen05.st (64 bf16 = 32 packed registers), operand B is a K-major tile of X by TMA.  Per K block the
// shared memory then carries 80 KB (32 KB of X written and read, 8 KB of codes written and read) instead of the
// 128 KB of the layout above.  Tensor memory: columns 0..255 the accumulator, 256..383 its copy rounded to
// bfloat16, 384..511 four A stages of 32 columns: there is no room for a second accumulator, so the epilogue first
// parks the rounded accumulator in the copy (fast: tensor memory to registers and back), releases the accumulator
// to the MMA, and writes the copy out beside the next tile's main loop.
// Warp roles: 0 TMA producer (X tiles and codes), 1 MMA issuer and tensor-memory owner, 4-7 and 12-15 two
// converter groups that take alternate K blocks (a warp reaches the lane quarter warp % 4), 8-11 epilogue.
struct FwdSmem {
  static constexpr int kBBytes = kTileN * kBK * 2;             // 32 KB of X
  static constexpr int kStages = 5;
  static constexpr int kRawBytes = kTileM * kBK;               // 8 KB of codes
  static constexpr int kRawStages = 4;
  static constexpr int kAStages = 4, kACols = kBK / 2;         // tensor-memory stages of A, 32 columns each
  static constexpr int kCopyCol = kTileN;                      // tensor-memory columns of the accumulator's bf16 copy
  static constexpr int kACol0 = kCopyCol + kTileN / 2;         // ... and of the first A stage
  static_assert(kACol0 + kAStages * kACols <= 512, "tensor memory columns");
  // per epilogue warp: a 32 x 32 bf16 block on its way to being stored transposed (rows of 64 bytes)
  static constexpr int kTransRow = 64, kTransBytes = 32 * kTransRow;
  static constexpr int kTransOffset = kStages * kBBytes + kRawStages * kRawBytes;
  static constexpr int kBarOffset = kTransOffset + 4 * kTransBytes;
  static constexpr int kBytes = kBarOffset + 512 + 1024;
  static constexpr int kThreads = 512;
};

__global__ void __launch_bounds__(FwdSmem::kThreads, 1)
int8_linear_forward_kernel(const __grid_constant__ LinArgs a, int32_t* __restrict__ status) {
  using S = FwdSmem;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* b_base = smem;
  uint8_t* raw_base = smem + S::kStages * S::kBBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::kBarOffset);
  uint64_t* b_full = bars;
  uint64_t* b_empty = b_full + S::kStages;
  uint64_t* raw_full = b_empty + S::kStages;
  uint64_t* raw_empty = raw_full + S::kRawStages;
  uint64_t* a_full = raw_empty + S::kRawStages;
  uint64_t* a_empty = a_full + S::kAStages;
  uint64_t* acc_full = a_empty + S::kAStages;
  uint64_t* acc_empty = acc_full + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < S::kStages; ++i) { mbar_init(&b_full[i], 1); mbar_init(&b_empty[i], 1); }
    for (int i = 0; i < S::kRawStages; ++i) { mbar_init(&raw_full[i], 1); mbar_init(&raw_empty[i], 4); }
    for (int i = 0; i < S::kAStages; ++i) { mbar_init(&a_full[i], 4); mbar_init(&a_empty[i], 1); }
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, 4);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_a = tmem_base + S::kACol0;

  // here a.rows / a.mblocks count rows of W (the accumulator's rows), a.cols / a.nblocks rows of X (its columns);
  // consecutive tiles (concurrent CTAs) share the block of X
  const int total = a.mblocks * a.nblocks;
  const int kblocks = (a.K + kBK - 1) / kBK;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer: X tile and codes
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < total; t += gridDim.x) {
        const int m0 = (t % a.mblocks) * kTileM, n0 = (t / a.mblocks) * kTileN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int rs = it % S::kRawStages, s = it % S::kStages;
          if (!mbar_wait(&raw_empty[rs], ((it / S::kRawStages) & 1) ^ 1)) { ok = false; break; }
          mbar_arrive_expect_tx(&raw_full[rs], S::kRawBytes);
          tma_load_2d(raw_base + rs * S::kRawBytes, &a.mapB, &raw_full[rs], kb * kBK, m0);
          if (!mbar_wait(&b_empty[s], ((it / S::kStages) & 1) ^ 1)) { ok = false; break; }
          mbar_arrive_expect_tx(&b_full[s], S::kBBytes);
          tma_load_2d(b_base + s * S::kBBytes, &a.mapA, &b_full[s], kb * kBK, n0);
        }
      }
      if (!ok) raise_expired(status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kTileM, kTileN, false, false);
      const uint64_t desc_b0 = umma_smem_desc_sw128(smem_u32(b_base), 16, 1024);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < total; t += gridDim.x, ++tcount) {
        if (!mbar_wait(acc_empty, (tcount & 1) ^ 1)) { ok = false; break; }
        tc_fence_after_sync();
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages, as = it % S::kAStages;
          if (!mbar_wait(&b_full[s], (it / S::kStages) & 1) || !mbar_wait(&a_full[as], (it / S::kAStages) & 1)) { ok = false; break; }
          tc_fence_after_sync();
          const uint64_t db = desc_b0 + (uint64_t)((s * S::kBBytes) >> 4);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            umma_bf16_tmem_a(tmem_base, tmem_a + as * S::kACols + k * 8, db + k * (32 >> 4), idesc, (kb | k) != 0);
          umma_commit(&b_empty[s]);
          umma_commit(&a_empty[as]);
        }
        if (ok) umma_commit(acc_full);
      }
      if (!ok) raise_expired(status);
    }
  } else if (warp >= 8 && warp < 12) {
    // ------------------------------------------------------------------ epilogue: row i of the tile is row m0 + i of W,
    // column c is row n0 + c of X.  A thread holds one row of the tile; each 32 x 32 block goes through shared
    // memory so that four lanes together store the 64 contiguous bytes it holds of one row of Y (2-byte stores,
    // 256 per thread and tile, took longer than the main loop of a short K; 16-byte stores to 32 different rows
    // per instruction flooded L2 with half-sector writes)
    const int q = warp & 3;
    uint8_t* trans = smem + S::kTransOffset + q * S::kTransBytes;
    uint32_t tcount = 0;
    bool ok = true;
    for (int t = blockIdx.x; ok && t < total; t += gridDim.x, ++tcount) {
      const int m0 = (t % a.mblocks) * kTileM, n0 = (t / a.mblocks) * kTileN;
      if (!mbar_wait(acc_full, tcount & 1)) { ok = false; break; }
      tc_fence_after_sync();
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16), tcopy = tacc + S::kCopyCol;
      // Phase 1: the accumulator is rounded to bfloat16 and parked in 128 spare columns of tensor memory, 32
      // columns at a time with the next load in flight; then the MMA may start the next tile.
      {
        uint32_t va[32], vb[32];
        auto park = [&](int c, const uint32_t* v) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
            pk[i] = *reinterpret_cast<uint32_t*>(&h);
          }
          tmem_st_32x16(tcopy + 16 * c, pk);
        };
        tmem_ld_32x32(tacc, va);
#pragma unroll 1
        for (int c = 0; c < kTileN / 32; c += 2) {
          tmem_ld_wait();
          tmem_ld_32x32(tacc + 32 * (c + 1), vb);
          park(c, va);
          tmem_ld_wait();
          if (c + 2 < kTileN / 32) tmem_ld_32x32(tacc + 32 * (c + 2), va);
          park(c + 1, vb);
        }
        tmem_st_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty);
      }
      // Phase 2, beside the next tile's main loop: the copy leaves through shared memory, transposed.
      auto emit = [&](int c, const uint32_t* pk) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {                   // block[j][lane] = D[lane][j], columns 2i and 2i + 1 in pk[i]
          *reinterpret_cast<uint16_t*>(trans + (2 * i) * S::kTransRow + lane * 2) = (uint16_t)(pk[i] & 0xFFFFu);
          *reinterpret_cast<uint16_t*>(trans + (2 * i + 1) * S::kTransRow + lane * 2) = (uint16_t)(pk[i] >> 16);
        }
        __syncwarp();
        const int piece = lane & 3, w0 = m0 + q * 32 + 8 * piece;   // this lane's 8 values of a row of Y start at w0
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int j = (lane >> 2) + 8 * i, tok = n0 + 32 * c + j;
          if (tok >= a.cols) continue;
          const uint4 val = *reinterpret_cast<const uint4*>(trans + j * S::kTransRow + 16 * piece);
          uint16_t* y = a.D + (int64_t)tok * a.ldd + w0;
          if (w0 + 8 <= a.rows) {
            *reinterpret_cast<uint4*>(y) = val;
          } else {
            const uint32_t w[4] = {val.x, val.y, val.z, val.w};
#pragma unroll
            for (int e = 0; e < 8; ++e)
              if (w0 + e < a.rows) y[e] = (uint16_t)((e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu));
          }
        }
        __syncwarp();
      };
      uint32_t pa[16], pb[16];
      tmem_ld_32x16(tcopy, pa);
#pragma unroll 1
      for (int c = 0; c < kTileN / 32; c += 2) {
        tmem_ld_wait();
        tmem_ld_32x16(tcopy + 16 * (c + 1), pb);
        emit(c, pa);
        tmem_ld_wait();
        if (c + 2 < kTileN / 32) tmem_ld_32x16(tcopy + 16 * (c + 2), pa);
        emit(c + 1, pb);
      }
    }
    if (!ok && lane == 0) raise_expired(status);
  } else if ((warp >= 4 && warp < 8) || warp >= 12) {
    // ------------------------------------------------------------------ converters: codes -> bf16 rows of A in tensor memory
    const int grp = warp >= 12 ? 1 : 0, q = warp & 3;
    const int row = q * 32 + lane;                       // row of the tile = lane of tensor memory
    uint32_t it = 0;
    bool ok = true;
    for (int t = blockIdx.x; ok && t < total; t += gridDim.x) {
      const int wr = (t % a.mblocks) * kTileM + row;
      const bool valid = wr < a.w_rows;
      for (int kb = 0; kb < kblocks; ++kb, ++it) {
        if ((int)(it & 1) != grp) continue;
        const int64_t idx = (int64_t)wr * a.ngroups + (kb >> 2);
        const float sc = valid ? __ldg(a.scales + idx) : 0.f;
        const float bias = 8388736.0f + (valid ? __ldg(a.zeros + idx) : 0.f);      // 2^23 + 128 + z
        const int rs = it % S::kRawStages, as = it % S::kAStages;
        if (!mbar_wait(&raw_full[rs], (it / S::kRawStages) & 1) || !mbar_wait(&a_empty[as], ((it / S::kAStages) & 1) ^ 1)) { ok = false; break; }
        tc_fence_after_sync();
        // codes: [128 rows][64 bytes], 16-byte piece c of row r stored at c ^ ((r >> 1) & 3)
        const uint8_t* rrow = raw_base + rs * S::kRawBytes + row * 64;
        uint32_t packed[32];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const uint4 codes = *reinterpret_cast<const uint4*>(rrow + ((c ^ ((row >> 1) & 3)) << 4));
          uint4 lo, hi;
          dequant16(codes, bias, sc, lo, hi);
          packed[8 * c + 0] = lo.x; packed[8 * c + 1] = lo.y; packed[8 * c + 2] = lo.z; packed[8 * c + 3] = lo.w;
          packed[8 * c + 4] = hi.x; packed[8 * c + 5] = hi.y; packed[8 * c + 6] = hi.z; packed[8 * c + 7] = hi.w;
        }
        tmem_st_32x32(tmem_a + ((uint32_t)(q * 32) << 16) + as * S::kACols, packed);
        tmem_st_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) { mbar_arrive(&a_full[as]); mbar_arrive(&raw_empty[rs]); }
      }
    }
    if (!ok && lane == 0) raise_expired(status);
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

int device_sms() {
  static int n = [] {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) v = 0;
    (void)cudaGetLastError();
    return v;
  }();
  return n > 0 ? n : 148;
}

template <int MODE>
int launch_mode(const LinArgs& args, int32_t* status, cudaStream_t st) {
  using S = LinSmem<MODE>;
  auto kern = int8_linear_kernel<MODE>;
  static bool smem_set[64] = {};                     // opted into its shared memory, per device
  int dev = 0;
  QG_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return QG_UNSUPPORTED_SHAPE;
  if (!smem_set[dev]) {
    QG_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kBytes));
    smem_set[dev] = true;
  }
  const int total = args.mblocks * args.nblocks;
  const int sms = device_sms();
  kern<<<total < sms ? total : sms, S::kThreads, S::kBytes, st>>>(args, status);
  QG_LAUNCH_CHECK();
  return QG_OK;
}

}  // namespace

int launch_int8_linear(int mode, const uint16_t* act, int64_t ld_act, const uint16_t* act2, int64_t ld_act2,
                       const qg_qtensor* W, int64_t T, int64_t m, int64_t n, uint16_t* D, int64_t ldd,
                       int32_t* status, cudaStream_t st) {
  LinArgs a;
  memset(&a, 0, sizeof(a));
  a.D = D;
  a.ldd = ldd;
  bool ok = true;
  if (mode == kWeightGrad) {
    // act = dY (T x m), act2 = X (T x n); both enter as 64-wide column slabs, K = T runs down the rows
    ok &= make_map_chunked(&a.mapA, act, T, (m + 63) / 64, ld_act, kBK, 2);
    ok &= make_map_chunked(&a.mapB, act2, T, (n + 63) / 64, ld_act2, kBK, 4);
    a.rows = (int32_t)m; a.cols = (int32_t)n; a.K = (int32_t)T;
  } else {
    a.scales = W->scales;
    a.zeros = W->zeros;
    a.ngroups = (int32_t)((n + kGroup - 1) / kGroup);
    a.w_rows = (int32_t)m;
    if (mode == kForward) {
      // the product is computed transposed: rows of the accumulator are rows of W, its columns rows of X
      ok &= make_map(&a.mapA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, act, n, T, ld_act, kBK, kTileN, CU_TENSOR_MAP_SWIZZLE_128B);
      ok &= make_map(&a.mapB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, W->codes, n, m, W->ld, kBK, kTileM, CU_TENSOR_MAP_SWIZZLE_64B);
      a.rows = (int32_t)m; a.cols = (int32_t)T; a.K = (int32_t)n;
    } else {
      // act = dY (T x m)
      ok &= make_map(&a.mapA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, act, m, T, ld_act, kBK, kTileM, CU_TENSOR_MAP_SWIZZLE_128B);
      ok &= make_map(&a.mapB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, W->codes, n, m, W->ld, kTileN, kBK, CU_TENSOR_MAP_SWIZZLE_NONE);
      a.rows = (int32_t)T; a.cols = (int32_t)n; a.K = (int32_t)m;
    }
  }
  if (!ok) return QG_CUDA_ERROR;
  // tiles per column of tiles: the input gradient's tiles are two row blocks high
  const int tile_rows = mode == kInputGrad ? LinSmem<kInputGrad>::kMT * kTileM : kTileM;
  a.mblocks = (a.rows + tile_rows - 1) / tile_rows;
  a.nblocks = (a.cols + kTileN - 1) / kTileN;
  if ((int64_t)a.mblocks * a.nblocks > (int64_t)1 << 30) return QG_UNSUPPORTED_SHAPE;   // the tile index is an int
  if (mode == kForward) {
    QG_CUDA_TRY(cudaFuncSetAttribute(int8_linear_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem::kBytes));
    const int total = a.mblocks * a.nblocks, sms = device_sms();
    int8_linear_forward_kernel<<<total < sms ? total : sms, FwdSmem::kThreads, FwdSmem::kBytes, st>>>(a, status);
    QG_LAUNCH_CHECK();
    return QG_OK;
  }
  return mode == kInputGrad ? launch_mode<kInputGrad>(a, status, st) : launch_mode<kWeightGrad>(a, status, st);
}

}  // namespace qg
