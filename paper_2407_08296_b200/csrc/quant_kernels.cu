// Stream kernels of the block-wise quantizer (Sec. 3.1, Sec. 3.3) and of the similarity
// statistic between adjacent projection matrices (Sec. 3.2).  All are HBM-bound: one warp
// owns one 256-element group, each lane eight consecutive elements (two 16-byte loads, one
// 8- or 4-byte store), the group minimum/maximum come from warp shuffles.
#include "qg_common.cuh"

namespace qg {

// ------------------------------------------------------------------------ quantize (RTN)
template <int BITS>
__global__ void __launch_bounds__(256)
quantize_rtn_kernel(const float* __restrict__ src, int64_t ld_src, int64_t rows, int64_t cols,
                    uint8_t* __restrict__ codes, int64_t ld_code_bytes,
                    float* __restrict__ scales, float* __restrict__ zeros, int ngroups) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (warp >= rows * ngroups) return;               // whole warps leave together
  const int64_t row = warp / ngroups;
  const int g = (int)(warp % ngroups);
  const int64_t c0 = (int64_t)g * kGroup + lane * 8;
  const int nvalid = (int)max((int64_t)0, min((int64_t)8, cols - c0));
  const float* p = src + row * ld_src + c0;

  float v[8];
  if (nvalid == 8) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p));
    const float4 b = __ldg(reinterpret_cast<const float4*>(p + 4));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = (i < nvalid) ? __ldg(p + i) : 0.0f;
  }
  float mn = INFINITY, mx = -INFINITY;
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (i < nvalid) { mn = fminf(mn, v[i]); mx = fmaxf(mx, v[i]); }
  mn = warp_min(mn);
  mx = warp_max(mx);
  const GroupParams gp = group_params<BITS>(mn, mx);
  if (lane == 0) {
    scales[row * ngroups + g] = gp.s;
    zeros[row * ngroups + g] = gp.z;
  }
  if (nvalid == 0) return;

  int q[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) q[i] = (i < nvalid) ? (int)rtn_code<BITS>(v[i], gp) : 0;

  if (BITS == 8) {
    uint8_t* out = codes + row * ld_code_bytes + c0;
    if (nvalid == 8) {
      uint2 w;
      w.x = (uint32_t)(q[0] & 0xFF) | ((uint32_t)(q[1] & 0xFF) << 8) | ((uint32_t)(q[2] & 0xFF) << 16) |
            ((uint32_t)(q[3] & 0xFF) << 24);
      w.y = (uint32_t)(q[4] & 0xFF) | ((uint32_t)(q[5] & 0xFF) << 8) | ((uint32_t)(q[6] & 0xFF) << 16) |
            ((uint32_t)(q[7] & 0xFF) << 24);
      *reinterpret_cast<uint2*>(out) = w;
    } else {
      for (int i = 0; i < nvalid; ++i) out[i] = (uint8_t)(q[i] & 0xFF);
    }
  } else if (BITS == 4) {
    uint8_t* out = codes + row * ld_code_bytes + (c0 >> 1);
    uint32_t w = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) w |= (uint32_t)((q[i] + 8) & 0xF) << (4 * i);   // padding nibbles hold code 0
    if (nvalid == 8) {
      *reinterpret_cast<uint32_t*>(out) = w;
    } else {
      for (int i = 0; i < (nvalid + 1) / 2; ++i) out[i] = (uint8_t)((w >> (8 * i)) & 0xFF);
    }
  } else {
    uint8_t* out = codes + row * ld_code_bytes + (c0 >> 2);
    uint32_t w = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) w |= (uint32_t)(((i < nvalid ? q[i] : 0) + 2) & 0x3) << (2 * i);   // padding holds code 0
    if (nvalid == 8) {
      *reinterpret_cast<uint16_t*>(out) = (uint16_t)w;
    } else {
      for (int i = 0; i < (nvalid + 3) / 4; ++i) out[i] = (uint8_t)((w >> (8 * i)) & 0xFF);
    }
  }
}

int launch_quantize_rtn(int bits, const float* src, int64_t rows, int64_t cols, int64_t ld_src,
                        const qg_qtensor* dst, cudaStream_t st) {
  const int ngroups = (int)ceil_div(cols, kGroup);
  const int64_t warps = rows * ngroups;
  const int64_t blocks = ceil_div(warps, 8);
  if (blocks > 0x7FFFFFFFll) return QG_UNSUPPORTED_SHAPE;
  if (bits == 8) {
    quantize_rtn_kernel<8><<<(unsigned)blocks, 256, 0, st>>>(src, ld_src, rows, cols, (uint8_t*)dst->codes, dst->ld,
                                                             dst->scales, dst->zeros, ngroups);
  } else if (bits == 4) {
    quantize_rtn_kernel<4><<<(unsigned)blocks, 256, 0, st>>>(src, ld_src, rows, cols, (uint8_t*)dst->codes,
                                                             dst->ld / 2, dst->scales, dst->zeros, ngroups);
  } else {
    quantize_rtn_kernel<2><<<(unsigned)blocks, 256, 0, st>>>(src, ld_src, rows, cols, (uint8_t*)dst->codes,
                                                             dst->ld / 4, dst->scales, dst->zeros, ngroups);
  }
  QG_LAUNCH_CHECK();
  return QG_OK;
}

// ------------------------------------------------------------------------ dequantize
__global__ void __launch_bounds__(256)
dequantize_kernel(qg_qtensor T, int ngroups, float* __restrict__ dst, int64_t ld_dst) {
  const int64_t chunks_per_row = ceil_div(T.cols, 8);
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T.rows * chunks_per_row) return;
  const int64_t row = idx / chunks_per_row;
  const int64_t c0 = (idx % chunks_per_row) * 8;
  const int nvalid = (int)min((int64_t)8, T.cols - c0);
  const int g = (int)(c0 / kGroup);
  const float s = __ldg(T.scales + row * ngroups + g), z = __ldg(T.zeros + row * ngroups + g);
  float q[8];
  load_codes8(T, row, c0, nvalid, q);
  float* out = dst + row * ld_dst + c0;
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (i < nvalid) out[i] = __fmul_rn(__fsub_rn(q[i], z), s);
}

int launch_dequantize(const qg_qtensor* src, float* dst, int64_t ld_dst, cudaStream_t st) {
  const int ngroups = (int)ceil_div(src->cols, kGroup);
  const int64_t threads = src->rows * ceil_div(src->cols, 8);
  const int64_t blocks = ceil_div(threads, 256);
  if (blocks > 0x7FFFFFFFll) return QG_UNSUPPORTED_SHAPE;
  dequantize_kernel<<<(unsigned)blocks, 256, 0, st>>>(*src, ngroups, dst, ld_dst);
  QG_LAUNCH_CHECK();
  return QG_OK;
}

// ------------------------------------------------------------------------ similarity (Sec. 3.2)
// Stage 1: each block takes kSimRows rows and all leading c columns (thread t: columns 8t..8t+7),
// accumulates the column dot products <a_j, b_j> over its rows and the two squared norms, and
// writes them to partial[block][...].  Stage 2 (one block) adds the partials in a fixed order,
// takes |.| per column and reduces with warp shuffles.  Deterministic: no atomics.
constexpr int kSimRows = 32;

__device__ __forceinline__ void load_p8(const qg_qtensor& T, int64_t row, int64_t c0, int ngroups, int nvalid,
                                        float v[8]) {
  const int g = (int)(c0 / kGroup);
  const float s = __ldg(T.scales + row * ngroups + g), z = __ldg(T.zeros + row * ngroups + g);
  float q[8];
  load_codes8(T, row, c0, nvalid, q);
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = (i < nvalid) ? __fmul_rn(__fsub_rn(q[i], z), s) : 0.0f;
}

__global__ void __launch_bounds__(256)
similarity_partial_kernel(qg_qtensor A, qg_qtensor B, int c, int c_pad, float* __restrict__ partial) {
  const int ngroups = (int)((A.cols + kGroup - 1) / kGroup);
  const int64_t row0 = (int64_t)blockIdx.x * kSimRows;
  const int64_t row1 = min(A.rows, row0 + kSimRows);
  float* out = partial + (int64_t)blockIdx.x * (c_pad + 2);
  float na = 0.f, nb = 0.f;
  for (int c0 = threadIdx.x * 8; c0 < c_pad; c0 += blockDim.x * 8) {
    const int nvalid = max(0, min(8, c - c0));
    float dot[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (nvalid > 0) {
      for (int64_t row = row0; row < row1; ++row) {
        float a[8], b[8];
        load_p8(A, row, c0, ngroups, nvalid, a);
        load_p8(B, row, c0, ngroups, nvalid, b);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          dot[i] = fmaf(a[i], b[i], dot[i]);
          na = fmaf(a[i], a[i], na);
          nb = fmaf(b[i], b[i], nb);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) out[c0 + i] = dot[i];
  }
  __shared__ float s_na[8], s_nb[8];
  na = warp_sum(na);
  nb = warp_sum(nb);
  if ((threadIdx.x & 31) == 0) { s_na[threadIdx.x >> 5] = na; s_nb[threadIdx.x >> 5] = nb; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float ta = 0.f, tb = 0.f;
    for (int w = 0; w < 8; ++w) { ta += s_na[w]; tb += s_nb[w]; }
    out[c_pad] = ta;
    out[c_pad + 1] = tb;
  }
}

__global__ void __launch_bounds__(1024)
similarity_final_kernel(const float* __restrict__ partial, int nblocks, int c, int c_pad, float* __restrict__ sim) {
  double num = 0.0, na = 0.0, nb = 0.0;
  for (int j = threadIdx.x; j < c; j += blockDim.x) {
    double d = 0.0;
    for (int b = 0; b < nblocks; ++b) d += (double)partial[(int64_t)b * (c_pad + 2) + j];
    num += fabs(d);
  }
  for (int b = threadIdx.x; b < nblocks; b += blockDim.x) {
    na += (double)partial[(int64_t)b * (c_pad + 2) + c_pad];
    nb += (double)partial[(int64_t)b * (c_pad + 2) + c_pad + 1];
  }
  __shared__ double s[3][32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    num += __shfl_xor_sync(0xFFFFFFFFu, num, o);
    na += __shfl_xor_sync(0xFFFFFFFFu, na, o);
    nb += __shfl_xor_sync(0xFFFFFFFFu, nb, o);
  }
  if ((threadIdx.x & 31) == 0) {
    s[0][threadIdx.x >> 5] = num; s[1][threadIdx.x >> 5] = na; s[2][threadIdx.x >> 5] = nb;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double tn = 0, ta = 0, tb = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { tn += s[0][w]; ta += s[1][w]; tb += s[2][w]; }
    const double den = sqrt(ta) * sqrt(tb);
    *sim = den > 0.0 ? (float)(tn / den) : 0.0f;
  }
}

size_t similarity_workspace_bytes(int64_t rows, int64_t cols) {
  const int64_t nblocks = ceil_div(rows, kSimRows);
  return (size_t)(nblocks * (round_up(cols, 8) + 2)) * sizeof(float);
}

int launch_similarity(const qg_qtensor* A, const qg_qtensor* B, int32_t c, float* sim_dev, void* ws,
                      cudaStream_t st) {
  const int nblocks = (int)ceil_div(A->rows, kSimRows);
  const int c_pad = (int)round_up(c, 8);
  similarity_partial_kernel<<<nblocks, 256, 0, st>>>(*A, *B, c, c_pad, (float*)ws);
  QG_LAUNCH_CHECK();
  similarity_final_kernel<<<1, 1024, 0, st>>>((const float*)ws, nblocks, c, c_pad, sim_dev);
  QG_LAUNCH_CHECK();
  return QG_OK;
}

}  // namespace qg

// ------------------------------------------------------------------------ similarity without a caller workspace
// The scratch of the two similarity kernels lives in this fixed device array instead of memory the
// caller allocates.  Every device that loads the library carries these 2 MiB until the process exits.
namespace {
constexpr size_t kStaticSimilarityBytes = 2u << 20;
static __device__ __align__(256) unsigned char g_similarity_scratch[kStaticSimilarityBytes];
constexpr int kMaxDevices = 64;
void* g_similarity_scratch_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal
}  // namespace

extern "C" QG_API size_t qgalore_subspace_similarity_static_max_bytes(void) { return kStaticSimilarityBytes; }

extern "C" QG_API int qgalore_subspace_similarity_static(const qg_qtensor* A, const qg_qtensor* B, int32_t sim_cols,
                                                         float* sim_dev, void* stream) {
  using namespace qg;
  if (!sim_dev) return QG_INVALID_ARGUMENT;
  // exactly the rules of qgalore_subspace_similarity: what that entry point refuses, this one refuses too
  int rc = check_projection_qtensor(A);
  if (rc != QG_OK) return rc;
  rc = check_projection_qtensor(B);
  if (rc != QG_OK) return rc;
  if (A->rows != B->rows || A->cols != B->cols) return QG_INVALID_ARGUMENT;
  if (!aligned4(sim_dev)) return QG_MISALIGNED;
  if (A->cols > 16384) return QG_UNSUPPORTED_SHAPE;
  // the shape must fit the fixed array: report it as a workspace that cannot be made larger
  if (similarity_workspace_bytes(A->rows, A->cols) > kStaticSimilarityBytes) return QG_WORKSPACE_TOO_SMALL;
  int dev = 0;
  QG_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return QG_UNSUPPORTED_SHAPE;
  if (!g_similarity_scratch_ptr[dev]) {
    // In host code the array's name is only a handle; the kernels need its address on the current device.
    void* p = nullptr;
    QG_CUDA_TRY(cudaGetSymbolAddress(&p, g_similarity_scratch));
    g_similarity_scratch_ptr[dev] = p;
  }
  const int32_t c = (sim_cols <= 0 || sim_cols > A->cols) ? (int32_t)A->cols : sim_cols;
  // the first kernel overwrites every scratch word the second one reads, so nothing has to be cleared
  return launch_similarity(A, B, c, sim_dev, g_similarity_scratch_ptr[dev], (cudaStream_t)stream);
}
