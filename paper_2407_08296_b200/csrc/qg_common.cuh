// Shared host/device helpers of the Q-GaLore library: status plumbing, launch accounting and
// the small device routines every kernel uses (Philox4x32-10, group parameters of the
// block-wise quantizer, bfloat16 conversion, INT4/INT8 unpacking).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <float.h>
#include <stdint.h>

#define QGALORE_TEST_API            // the library implements the test aids the header guards
#include "../../include/qgalore.h"

namespace qg {

constexpr int kGroup = 256;  // Sec. 3.1: block size 256

// Bumped whenever a change to the step's kernels can move their DRAM traffic or timing (see qgalore_kernel_revision).
#define QG_STEP_KERNELS_REVISION "step-2026-11-30a"

// ----------------------------------------------------------------------------- host plumbing
void note_cuda_error(cudaError_t e, const char* where);
void count_launch(int n = 1);

#define QG_CUDA_TRY(expr)                                  \
  do {                                                     \
    cudaError_t qg_e_ = (expr);                            \
    if (qg_e_ != cudaSuccess) {                            \
      ::qg::note_cuda_error(qg_e_, #expr);                 \
      return QG_CUDA_ERROR;                                \
    }                                                      \
  } while (0)

#define QG_LAUNCH_CHECK()                                  \
  do {                                                     \
    ::qg::count_launch();                                  \
    cudaError_t qg_e_ = cudaPeekAtLastError();             \
    if (qg_e_ != cudaSuccess) {                            \
      ::qg::note_cuda_error(qg_e_, "kernel launch");       \
      return QG_CUDA_ERROR;                                \
    }                                                      \
  } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

// Pointer, extent and alignment rules of a quantized matrix that every entry point applies: non-null buffers,
// positive extents, pitch >= cols, the expected code width, groups of 256; codes 16-byte aligned with rows of
// whole 16-byte units, scales and zero points 4-byte aligned (the kernels read them as binary32 words).
inline int check_qtensor(const qg_qtensor* t, int bits) {
  if (!t || !t->codes || !t->scales || !t->zeros) return QG_INVALID_ARGUMENT;
  if (t->rows <= 0 || t->cols <= 0 || t->ld < t->cols) return QG_INVALID_ARGUMENT;
  if (t->bits != bits || t->group != 256) return QG_INVALID_ARGUMENT;
  if (!aligned16(t->codes) || !aligned4(t->scales) || !aligned4(t->zeros)) return QG_MISALIGNED;
  if (t->ld % (128 / bits) != 0) return QG_MISALIGNED;      // a row of codes is a multiple of 16 bytes
  return QG_OK;
}
// The same for a projection matrix, whose codes may be 2, 4 or 8 bits wide (Sec. 4.4, Fig. 3).
inline int check_projection_qtensor(const qg_qtensor* t) {
  if (!t || (t->bits != 2 && t->bits != 4 && t->bits != 8)) return QG_INVALID_ARGUMENT;
  return check_qtensor(t, t->bits);
}
#ifdef __CUDACC__
#define QG_HD __host__ __device__
#else
#define QG_HD
#endif
QG_HD inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
QG_HD inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }

// Scalars of one step as the kernels take them.
struct StepScalars {
  float beta1, beta2, one_minus_beta1, one_minus_beta2;
  float bias1, bias2;      // 1 - beta^t, computed in double on the host
  float eps;
  float lr_alpha;          // lr * alpha
  float lr_wd;             // lr * weight_decay
  uint32_t seed_lo, seed_hi, step_lo, step_hi;
  int32_t rounding;        // QG_ROUND_STOCHASTIC or QG_ROUND_NEAREST
};

// ----------------------------------------------------------------------------- device helpers
#ifdef __CUDACC__

// Philox4x32 with 10 rounds (Salmon et al., SC'11).
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}

// The eight 16-bit uniforms of columns 8*blk .. 8*blk+7 of row `row`: lane l of the block is
// bits [16*(l&1), +16) of output word l>>1.
__device__ __forceinline__ void sr_lanes8(const StepScalars& sc, uint32_t row, uint32_t blk, float h[8]) {
  const uint4 x = philox4x32_10(make_uint4(blk, row, sc.step_lo, sc.step_hi), make_uint2(sc.seed_lo, sc.seed_hi));
  h[0] = (float)(x.x & 0xFFFFu); h[1] = (float)(x.x >> 16);
  h[2] = (float)(x.y & 0xFFFFu); h[3] = (float)(x.y >> 16);
  h[4] = (float)(x.z & 0xFFFFu); h[5] = (float)(x.z >> 16);
  h[6] = (float)(x.w & 0xFFFFu); h[7] = (float)(x.w >> 16);
}

struct GroupParams { float s, inv, z; };

// Scale, reciprocal and zero point of one group from its minimum and maximum (Sec. 3.1):
// s = (max - min) / (2^bits - 1) in binary32, inv = 1 / s, z = -2^(bits-1) - rint(min * inv).
// A constant group, or one whose s is not a normal number, takes z = 0 and s = |max| (1 if
// that is not a normal number).  Every operation is a single correctly rounded binary32 one.
template <int BITS>
__device__ __forceinline__ GroupParams group_params(float mn, float mx) {
  constexpr float kLevels = (float)((1 << BITS) - 1);
  constexpr float kQlo = -(float)(1 << (BITS - 1));
  float s = __fdiv_rn(__fsub_rn(mx, mn), kLevels);
  const bool degenerate = (mx == mn) || !isfinite(s) || (s < FLT_MIN);
  if (degenerate) {
    const float amx = fabsf(mx);
    s = (isfinite(amx) && amx >= FLT_MIN) ? amx : 1.0f;
  }
  GroupParams g;
  g.s = s;
  g.inv = __fdiv_rn(1.0f, s);
  g.z = degenerate ? 0.0f : __fsub_rn(kQlo, rintf(__fmul_rn(mn, g.inv)));
  return g;
}

template <int BITS>
__device__ __forceinline__ float rtn_code(float x, const GroupParams& g) {
  constexpr float kQlo = -(float)(1 << (BITS - 1));
  constexpr float kQhi = (float)((1 << (BITS - 1)) - 1);
  const float q = __fadd_rn(rintf(__fmul_rn(x, g.inv)), g.z);
  return fminf(fmaxf(q, kQlo), kQhi);
}

// Stochastic rounding of the scaled value (Sec. 3.4): floor, plus one iff frac * 65536 > h.
__device__ __forceinline__ float sr_code(float x, const GroupParams& g, float h) {
  const float t = __fmul_rn(x, g.inv);
  const float f = floorf(t);
  const float frac = __fsub_rn(t, f);
  const float up = (__fmul_rn(frac, 65536.0f) > h) ? 1.0f : 0.0f;
  const float q = __fadd_rn(__fadd_rn(f, up), g.z);
  return fminf(fmaxf(q, -128.0f), 127.0f);
}

__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ uint16_t float_to_bf16_bits(float f) {
  return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

// Eight INT8 codes (one uint2) -> floats.
__device__ __forceinline__ void unpack_int8x8(uint2 w, float q[8]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    q[i] = (float)(int8_t)((w.x >> (8 * i)) & 0xFFu);
    q[4 + i] = (float)(int8_t)((w.y >> (8 * i)) & 0xFFu);
  }
}
// Eight INT4 codes (one uint32, stored as code + 8, low nibble first) -> floats in [-8, 7].
__device__ __forceinline__ void unpack_int4x8(uint32_t w, float q[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) q[i] = (float)((int)((w >> (4 * i)) & 0xFu) - 8);
}

// Eight INT2 codes (one uint16, stored as code + 2, column 8k + i in bits 2i, 2i + 1) -> floats in [-2, 1].
__device__ __forceinline__ void unpack_int2x8(uint32_t w, float q[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) q[i] = (float)((int)((w >> (2 * i)) & 0x3u) - 2);
}

// Bytes per row of codes and per eight codes, for the three widths the projection may take (Sec. 4.4, Fig. 3).
__device__ __forceinline__ int64_t code_row_bytes(const qg_qtensor& T) { return T.bits == 8 ? T.ld : (T.bits == 4 ? T.ld / 2 : T.ld / 4); }

// Codes of columns c0 .. c0 + 7 (c0 a multiple of 8) of a row as floats; the first nvalid are real.
__device__ __forceinline__ void load_codes8(const qg_qtensor& T, int64_t row, int64_t c0, int nvalid, float q[8]) {
  const uint8_t* base = (const uint8_t*)T.codes + row * code_row_bytes(T);
  if (T.bits == 8) {
    const uint8_t* p = base + c0;
    if (nvalid == 8) {
      unpack_int8x8(__ldg(reinterpret_cast<const uint2*>(p)), q);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) q[i] = (i < nvalid) ? (float)(int8_t)p[i] : 0.0f;
    }
  } else if (T.bits == 4) {
    const uint8_t* p = base + (c0 >> 1);
    uint32_t w = 0;
    if (nvalid == 8) {
      w = __ldg(reinterpret_cast<const uint32_t*>(p));
    } else {
      for (int i = 0; i < (nvalid + 1) / 2; ++i) w |= (uint32_t)p[i] << (8 * i);
    }
    unpack_int4x8(w, q);
  } else {
    const uint8_t* p = base + (c0 >> 2);
    uint32_t w = 0;
    if (nvalid == 8) {
      w = __ldg(reinterpret_cast<const uint16_t*>(p));
    } else {
      for (int i = 0; i < (nvalid + 3) / 4; ++i) w |= (uint32_t)p[i] << (8 * i);
    }
    unpack_int2x8(w, q);
  }
}

#endif  // __CUDACC__

// ----------------------------------------------------------------------------- kernel launchers
// quant_kernels.cu
int launch_quantize_rtn(int bits, const float* src, int64_t rows, int64_t cols, int64_t ld_src,
                        const qg_qtensor* dst, cudaStream_t st);
int launch_dequantize(const qg_qtensor* src, float* dst, int64_t ld_dst, cudaStream_t st);
int launch_similarity(const qg_qtensor* A, const qg_qtensor* B, int32_t c, float* sim_dev,
                      void* ws, cudaStream_t st);
size_t similarity_workspace_bytes(int64_t rows, int64_t cols);

// step_*.cu
struct StepArgs {
  const uint16_t* G; int64_t ldg, m, n, r;
  qg_qtensor P, W;
  float* M; float* V; int64_t ldmv;
  StepScalars sc;
  void* ws; size_t ws_bytes;
  int32_t* status;
  qg_debug dbg;
  int32_t right;           // 0: R = P^T G, P m x r, moments r x n;  1: R = G Q, Q n x r, moments kept as r x m
  int32_t state8;          // moments stored in 8 bits: M, V point to int8 / uint8 codes (pitch ldmv bytes) ...
  float* M_scale;          // ... with one fp32 scale per block of 32 columns of a row, dense [r][ceil(cols / 32)]
  float* V_scale;
};
// P~ = bf16((q - z) * s) of an INT4 matrix whose column count is a multiple of 32 (row pitch ld_out elements)
int launch_dequant_p(const qg_qtensor& P, uint16_t* out, int64_t ld_out, cudaStream_t st);


// refresh.cu: one matrix of a batched subspace refresh
struct RefreshJob {
  const uint16_t* G; int64_t ldg;
  uint64_t seed;
  const qg_qtensor* P_new;
  float* P_fp32;           // optional
};

// linear_tc.cu: the INT8 linear layer of App. A.  mode 0: D (T x m) = act (X, T x n) W~^T; mode 1: D (T x n) =
// act (dY, T x m) W~; mode 2: D (m x n) = act^T (dY, T x m) act2 (X, T x n), W unused.  All bf16, row-major.
int launch_int8_linear(int mode, const uint16_t* act, int64_t ld_act, const uint16_t* act2, int64_t ld_act2,
                       const qg_qtensor* W, int64_t T, int64_t m, int64_t n, uint16_t* D, int64_t ldd,
                       int32_t* status, cudaStream_t st);

}  // namespace qg
