// Element-wise halves of the Q-GaLore step (Sec. 3.5), shared by every GEMM kernel's epilogue:
// the Adam moment update on eight consecutive columns of the r x n low-rank state, and the
// dequantize-add of eight consecutive weight columns.
#pragma once

#include "qg_common.cuh"

namespace qg {

// Adam on eight consecutive elements (row i, columns j0..j0+7) of the low-rank state:
//   M <- b1 M + (1-b1) R,  V <- b2 V + (1-b2) R^2,  N = (M / bias1) / (sqrt(V / bias2) + eps)
// (Kingma & Ba; bias correction on, eps outside the root).  nvalid < 8 on the ragged edge.
__device__ __forceinline__ void adam8(const StepScalars& sc, const float r8[8], float* __restrict__ Mrow,
                                      float* __restrict__ Vrow, int nvalid, float n8[8]) {
  float m[8], v[8];
  if (nvalid == 8) {
    const float4 m0 = *reinterpret_cast<const float4*>(Mrow), m1 = *reinterpret_cast<const float4*>(Mrow + 4);
    const float4 v0 = *reinterpret_cast<const float4*>(Vrow), v1 = *reinterpret_cast<const float4*>(Vrow + 4);
    m[0] = m0.x; m[1] = m0.y; m[2] = m0.z; m[3] = m0.w; m[4] = m1.x; m[5] = m1.y; m[6] = m1.z; m[7] = m1.w;
    v[0] = v0.x; v[1] = v0.y; v[2] = v0.z; v[3] = v0.w; v[4] = v1.x; v[5] = v1.y; v[6] = v1.z; v[7] = v1.w;
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) { m[i] = (i < nvalid) ? Mrow[i] : 0.f; v[i] = (i < nvalid) ? Vrow[i] : 0.f; }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    m[i] = fmaf(sc.beta1, m[i], sc.one_minus_beta1 * r8[i]);
    v[i] = fmaf(sc.beta2, v[i], sc.one_minus_beta2 * r8[i] * r8[i]);
    n8[i] = (m[i] / sc.bias1) / (sqrtf(v[i] / sc.bias2) + sc.eps);
  }
  if (nvalid == 8) {
    *reinterpret_cast<float4*>(Mrow) = make_float4(m[0], m[1], m[2], m[3]);
    *reinterpret_cast<float4*>(Mrow + 4) = make_float4(m[4], m[5], m[6], m[7]);
    *reinterpret_cast<float4*>(Vrow) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(Vrow + 4) = make_float4(v[4], v[5], v[6], v[7]);
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (i < nvalid) { Mrow[i] = m[i]; Vrow[i] = v[i]; }
  }
}

__device__ __forceinline__ uint4 pack_bf16x8(const float f[8]) {
  uint4 o;
  o.x = (uint32_t)float_to_bf16_bits(f[0]) | ((uint32_t)float_to_bf16_bits(f[1]) << 16);
  o.y = (uint32_t)float_to_bf16_bits(f[2]) | ((uint32_t)float_to_bf16_bits(f[3]) << 16);
  o.z = (uint32_t)float_to_bf16_bits(f[4]) | ((uint32_t)float_to_bf16_bits(f[5]) << 16);
  o.w = (uint32_t)float_to_bf16_bits(f[6]) | ((uint32_t)float_to_bf16_bits(f[7]) << 16);
  return o;
}

__device__ __forceinline__ uint2 pack_int8x8(const float q[8]) {
  uint2 w;
  w.x = (uint32_t)((int)q[0] & 0xFF) | ((uint32_t)((int)q[1] & 0xFF) << 8) | ((uint32_t)((int)q[2] & 0xFF) << 16) |
        ((uint32_t)((int)q[3] & 0xFF) << 24);
  w.y = (uint32_t)((int)q[4] & 0xFF) | ((uint32_t)((int)q[5] & 0xFF) << 8) | ((uint32_t)((int)q[6] & 0xFF) << 16) |
        ((uint32_t)((int)q[7] & 0xFF) << 24);
  return w;
}

}  // namespace qg
