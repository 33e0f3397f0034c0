// Tensor-core products of the subspace refresh (Sec. 3.5): D (M x N, fp32) = A (M x K, bf16) * B (K x N, fp32).
//
// The two large products of a subspace iteration, Z = G^T Q and Y = G Z, have the gradient (bfloat16, exact) on one
// side and an fp32 iterate on the other.  The subspace next to the r-th singular value sits in the noise bulk of the
// gradient with relative gaps of 1e-4 .. 1e-3, so the products have to be fp32-faithful; bfloat16 operands are not.
// The iterate is therefore split into three bfloat16 planes, B = B_hi + B_mid + B_lo (each the bfloat16 rounding of
// what the planes before it leave: 3 x 8 significand bits, the residual is below 2^-24 of the element), and
//     A B = A B_hi + A B_mid + A B_lo
// is accumulated in fp32 in tensor memory by tcgen05.mma: every product of two bfloat16 values is exact, so the
// result carries the accumulation error of an fp32 dot product and nothing else.
//
// One persistent CTA per SM, tiles of 128 x 256, K blocks of 64.  A stage holds the A tile (16 KB) and the three B
// tiles (3 x 32 KB), all brought by TMA in the 128-byte swizzle; the MMA thread issues 3 x 4 instructions per stage
// into one of two accumulators, so that the fp32 epilogue of a tile overlaps the main loop of the next.  Warp roles:
// 0 TMA producer, 1 MMA issuer and tensor-memory owner, 4-7 epilogue.  A is read K-major (K contiguous: a 2-D map
// with exact bounds) or MN-major (M contiguous: 64-wide slabs through a 3-D view; the last slab may reach into the
// row padding of A, which only feeds output rows that are never written).
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
constexpr int kTileN = 256;    // accumulator columns
constexpr int kSlab = 64 * kBK * 2;   // one 64-wide MN-major slab of a stage: 64 K rows of 128 bytes
constexpr int kPlanes = 3;

struct SplitArgs {
  CUtensorMap mapA;            // bf16 A: K-major 2-D (box 64 x 128) or chunked 3-D (box 64 x 64 x 2)
  CUtensorMap mapB;            // the three planes of B stacked along K: chunked 3-D over [3 * kpad][N], box 64 x 64 x 4
  float* D;
  int64_t ldd;
  int32_t M, N, K, kpad;
  int32_t mblocks, nblocks;
};

struct SplitSmem {
  static constexpr int kABytes = kTileM * kBK * 2;             // 16 KB
  static constexpr int kBBytes = kTileN * kBK * 2;             // 32 KB per plane
  static constexpr int kStageBytes = kABytes + kPlanes * kBBytes;
  static constexpr int kStages = 2;
  static constexpr int kBarOffset = kStages * kStageBytes;
  static constexpr int kBytes = kBarOffset + 256 + 1024;       // barriers + slack for 1024-byte alignment
  static constexpr int kEpiWarps = 4;
  static constexpr int kThreads = (4 + kEpiWarps) * 32;
  static_assert(kBytes <= 227 * 1024, "shared memory budget");
};

__device__ __forceinline__ void raise_expired(int32_t* status) {
  if (status) atomicOr(status, QG_DEV_WAIT_EXPIRED);
}

template <bool A_MN>
__global__ void __launch_bounds__(SplitSmem::kThreads, 1)
split_gemm_kernel(const __grid_constant__ SplitArgs a, int32_t* __restrict__ status) {
  using S = SplitSmem;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stage_base = smem;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::kBarOffset);
  uint64_t* full = bars;
  uint64_t* empty = full + S::kStages;
  uint64_t* acc_full = empty + S::kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < S::kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], S::kEpiWarps); }
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // tile t -> (m block, n block): consecutive tiles (concurrent CTAs) share the n block, i.e. the same columns of
  // the three planes of B, which are then served from L2
  const int total = a.mblocks * a.nblocks;
  const int kblocks = (a.K + kBK - 1) / kBK;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < total; t += gridDim.x) {
        const int m0 = (t % a.mblocks) * kTileM, n0 = (t / a.mblocks) * kTileN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          if (!mbar_wait(&empty[s], ((it / S::kStages) & 1) ^ 1)) { ok = false; break; }
          uint8_t* sA = stage_base + s * S::kStageBytes;
          mbar_arrive_expect_tx(&full[s], S::kStageBytes);
          if (A_MN) tma_load_3d(sA, &a.mapA, &full[s], 0, kb * kBK, m0 / 64);
          else tma_load_2d(sA, &a.mapA, &full[s], kb * kBK, m0);
#pragma unroll
          for (int p = 0; p < kPlanes; ++p)
            tma_load_3d(sA + S::kABytes + p * S::kBBytes, &a.mapB, &full[s], 0, p * a.kpad + kb * kBK, n0 / 64);
        }
      }
      if (!ok) raise_expired(status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kTileM, kTileN, A_MN, true);
      // K-major: rows of 128 bytes, 8-row groups 1024 bytes apart, 16 K indices = 32 bytes along the row.
      // MN-major: 64-wide slabs of kSlab bytes, 8 K indices = 1024 bytes, 16 K indices = 2048 bytes.
      const uint64_t desc_a0 = A_MN ? umma_smem_desc_sw128(smem_u32(stage_base), kSlab, 1024)
                                    : umma_smem_desc_sw128(smem_u32(stage_base), 16, 1024);
      const uint64_t desc_b0 = umma_smem_desc_sw128(smem_u32(stage_base) + S::kABytes, kSlab, 1024);
      constexpr uint64_t astep = A_MN ? (2048 >> 4) : (32 >> 4);
      constexpr uint64_t bstep = 2048 >> 4;
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < total; t += gridDim.x, ++tcount) {
        const uint32_t ab = tcount & 1;
        if (!mbar_wait(&acc_empty[ab], ((tcount >> 1) & 1) ^ 1)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + ab * kTileN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % S::kStages;
          if (!mbar_wait(&full[s], (it / S::kStages) & 1)) { ok = false; break; }
          tc_fence_after_sync();
          const uint64_t da = desc_a0 + (uint64_t)((s * S::kStageBytes) >> 4);
          // the smallest plane first: the low-order terms are in the accumulator before the large ones arrive
#pragma unroll
          for (int p = kPlanes - 1; p >= 0; --p) {
            const uint64_t db = desc_b0 + (uint64_t)((s * S::kStageBytes + p * S::kBBytes) >> 4);
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)
              umma_bf16(d_tmem, da + k * astep, db + k * bstep, idesc, (kb != 0) || (p != kPlanes - 1) || (k != 0));
          }
          umma_commit(&empty[s]);
        }
        if (ok) umma_commit(&acc_full[ab]);
      }
      if (!ok) raise_expired(status);
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ epilogue: the fp32 accumulator as it is
    const int q = warp & 3;
    uint32_t tcount = 0;
    bool ok = true;
    for (int t = blockIdx.x; ok && t < total; t += gridDim.x, ++tcount) {
      const int m0 = (t % a.mblocks) * kTileM, n0 = (t / a.mblocks) * kTileN;
      const uint32_t ab = tcount & 1;
      if (!mbar_wait(&acc_full[ab], (tcount >> 1) & 1)) { ok = false; break; }
      tc_fence_after_sync();
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + ab * kTileN;
      const int row = m0 + q * 32 + lane;
      float* drow = a.D + (int64_t)row * a.ldd;
#pragma unroll 1
      for (int c = 0; c < kTileN / 32; ++c) {
        uint32_t v[32];
        tmem_ld_32x32(tacc + 32 * c, v);
        tmem_ld_wait();
        if (c == kTileN / 32 - 1) {                    // every read of this accumulator has landed
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&acc_empty[ab]);
        }
        const int col = n0 + 32 * c;
        if (row < a.M && col < a.N) {
          if (col + 32 <= a.N) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
              *reinterpret_cast<uint4*>(drow + col + 4 * i) = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (col + i < a.N) drow[col + i] = __uint_as_float(v[i]);
          }
        }
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

// B (K x N fp32, pitch ldb) -> three bfloat16 planes [kpad][N] each, stacked: hi = bf16(x), mid = bf16(x - hi),
// lo = bf16(x - hi - mid) (the subtractions are exact in binary32).  Rows K .. kpad - 1 are written as zero, so that
// a K block that reaches past K reads zeros and never the next plane.  A thread takes eight columns.
__global__ void __launch_bounds__(256)
split_planes_kernel(const float* __restrict__ B, int64_t ldb, int K, int N, int kpad, uint16_t* __restrict__ planes) {
  const int64_t per_row = N / 8;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)kpad * per_row) return;
  const int64_t row = idx / per_row, c0 = (idx - row * per_row) * 8;
  float x[8];
  if (row < K) {
    const float4 u = *reinterpret_cast<const float4*>(B + row * ldb + c0), w = *reinterpret_cast<const float4*>(B + row * ldb + c0 + 4);
    x[0] = u.x; x[1] = u.y; x[2] = u.z; x[3] = u.w; x[4] = w.x; x[5] = w.y; x[6] = w.z; x[7] = w.w;
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = 0.f;
  }
  uint32_t out[kPlanes][4];
#pragma unroll
  for (int i = 0; i < 8; i += 2) {
    float r0 = x[i], r1 = x[i + 1];
#pragma unroll
    for (int p = 0; p < kPlanes; ++p) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(r0, r1);
      out[p][i >> 1] = *reinterpret_cast<const uint32_t*>(&h);
      r0 = __fsub_rn(r0, __low2float(h));
      r1 = __fsub_rn(r1, __high2float(h));
    }
  }
#pragma unroll
  for (int p = 0; p < kPlanes; ++p)
    *reinterpret_cast<uint4*>(planes + ((int64_t)p * kpad + row) * N + c0) = make_uint4(out[p][0], out[p][1], out[p][2], out[p][3]);
}

int split_sm_count() {
  static int n = [] {
    int dev = 0, v = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    return v > 0 ? v : 148;
  }();
  return n;
}

}  // namespace

// Scratch the planes of a K x N iterate need.
size_t split_planes_bytes(int64_t K, int64_t N) { return (size_t)(kPlanes * round_up(K, kBK) * N * 2); }

// Whether a product of these extents and strides can take the tensor-core route (else the caller keeps the
// CUDA-core kernel): N a multiple of 64, A 16-byte aligned with a pitch of whole 16-byte units that, for the
// MN-major form, covers the last 64-wide slab of M.
bool split_gemm_supported(const uint16_t* A, int64_t sa_m, int64_t sa_k, int64_t M, int64_t N, int64_t K) {
  if (M <= 0 || N <= 0 || K <= 0 || N % 64 != 0 || M > (1ll << 30) || K > (1ll << 30)) return false;
  if ((reinterpret_cast<uintptr_t>(A) & 15u) != 0) return false;
  if (sa_k == 1) return sa_m % 8 == 0 && sa_m >= K;                       // K-major: rows of K contiguous elements
  if (sa_m == 1) return sa_k % 8 == 0 && sa_k >= round_up(M, 64);          // MN-major: rows of M contiguous elements
  return false;
}

// D (M x N fp32, pitch ldd) = A * B with A(i, k) = A[i * sa_m + k * sa_k] in bfloat16 and B (K x N fp32, pitch ldb)
// split into `planes` (split_planes_bytes(K, N) bytes of scratch) first.
int launch_split_gemm(const uint16_t* A, int64_t sa_m, int64_t sa_k, const float* B, int64_t ldb, float* D, int64_t ldd,
                      int64_t M, int64_t N, int64_t K, uint16_t* planes, int32_t* status, cudaStream_t st) {
  const int kpad = (int)round_up(K, kBK);
  {
    const int64_t threads = (int64_t)kpad * (N / 8);
    split_planes_kernel<<<(unsigned)ceil_div(threads, 256), 256, 0, st>>>(B, ldb, (int)K, (int)N, kpad, planes);
    QG_LAUNCH_CHECK();
  }
  SplitArgs a;
  memset(&a, 0, sizeof(a));
  const bool a_mn = sa_m == 1;
  bool ok = true;
  if (a_mn) ok &= make_map_chunked(&a.mapA, A, K, ceil_div(M, 64), sa_k, kBK, 2);
  else ok &= make_map(&a.mapA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, A, K, M, sa_m, kBK, kTileM, CU_TENSOR_MAP_SWIZZLE_128B);
  ok &= make_map_chunked(&a.mapB, planes, (int64_t)kPlanes * kpad, N / 64, N, kBK, kTileN / 64);
  if (!ok) {
    note_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled");
    return QG_CUDA_ERROR;
  }
  a.D = D; a.ldd = ldd;
  a.M = (int32_t)M; a.N = (int32_t)N; a.K = (int32_t)K; a.kpad = kpad;
  a.mblocks = (int32_t)ceil_div(M, kTileM);
  a.nblocks = (int32_t)ceil_div(N, kTileN);
  const int total = a.mblocks * a.nblocks;
  const int grid = total < split_sm_count() ? total : split_sm_count();
  static bool smem_set[2][64] = {};
  int dev = 0;
  QG_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return QG_UNSUPPORTED_SHAPE;
  if (a_mn) {
    if (!smem_set[1][dev]) {
      QG_CUDA_TRY(cudaFuncSetAttribute(split_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SplitSmem::kBytes));
      smem_set[1][dev] = true;
    }
    split_gemm_kernel<true><<<grid, SplitSmem::kThreads, SplitSmem::kBytes, st>>>(a, status);
  } else {
    if (!smem_set[0][dev]) {
      QG_CUDA_TRY(cudaFuncSetAttribute(split_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SplitSmem::kBytes));
      smem_set[0][dev] = true;
    }
    split_gemm_kernel<false><<<grid, SplitSmem::kThreads, SplitSmem::kBytes, st>>>(a, status);
  }
  QG_LAUNCH_CHECK();
  return QG_OK;
}

}  // namespace qg
