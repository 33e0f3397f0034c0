// CUDA-core version of the Q-GaLore step (Sec. 3.5): three launches per matrix,
//   (1) P~ = bf16(dequant(P))                                 -> workspace, m x r bf16
//   (2) R = P~^T G, Adam on (M, V), N_b = bf16(N)             -> workspace, r x n bf16
//   (3) D = P~ N_b, W' = dequant(W) - lr*alpha*D, Quant_8 with stochastic rounding, in place
// A 32 x 256 output tile per block of 256 threads: warp w owns rows 4w..4w+3, lane l the eight
// columns 8l..8l+7, so one warp holds one whole quantization group of a row and the group
// minimum/maximum are warp-shuffle reductions.  fp32 accumulation of bf16 products.
#include "step_epilogue.cuh"

namespace qg {

namespace {

constexpr int kTM = 32, kTN = 256, kTK = 32;

__global__ void __launch_bounds__(256)
dequant_p_bf16_kernel(qg_qtensor P, uint16_t* __restrict__ out, int64_t ld_out) {
  const int ngroups = (int)((P.cols + kGroup - 1) / kGroup);
  const int64_t chunks = P.cols / 8;                 // r % 32 == 0
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= P.rows * chunks) return;
  const int64_t row = idx / chunks, c0 = (idx % chunks) * 8;
  const int g = (int)(c0 / kGroup);
  const float s = __ldg(P.scales + row * ngroups + g), z = __ldg(P.zeros + row * ngroups + g);
  float q[8], v[8];
  load_codes8(P, row, c0, 8, q);                     // 2-, 4- or 8-bit codes
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __fmul_rn(__fsub_rn(q[i], z), s);
  *reinterpret_cast<uint4*>(out + row * ld_out + c0) = pack_bf16x8(v);
}

// C[MxN] = A * B with B[K][N] row-major bf16.  A_TRANS: A is stored [K][M] (element (i,k) at
// A[k*lda + i]); otherwise [M][K].  acc[4][8] per thread; the epilogue functor consumes it.
template <bool A_TRANS, class Epi>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const uint16_t* __restrict__ A, int64_t lda, const uint16_t* __restrict__ B, int64_t ldb,
                 int64_t Mdim, int64_t Ndim, int64_t Kdim, Epi epi) {
  __shared__ float As[kTK][kTM + 1];
  __shared__ __align__(16) uint16_t Bs[kTK][kTN];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t row0 = (int64_t)blockIdx.y * kTM, col0 = (int64_t)blockIdx.x * kTN;
  float acc[4][8];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  for (int64_t k0 = 0; k0 < Kdim; k0 += kTK) {
    // A tile: 32 x 32 elements, four per thread
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = tid + e * 256;
      int kk, ii;
      if (A_TRANS) { kk = idx >> 5; ii = idx & 31; } else { ii = idx >> 5; kk = idx & 31; }
      const int64_t gk = k0 + kk, gi = row0 + ii;
      float v = 0.f;
      if (gk < Kdim && gi < Mdim) v = bf16_bits_to_float(A_TRANS ? A[gk * lda + gi] : A[gi * lda + gk]);
      As[kk][ii] = v;
    }
    // B tile: 32 x 256 bf16 = 1024 16-byte vectors, four per thread
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = tid + e * 256;
      const int kk = idx >> 5, cv = (idx & 31) * 8;
      const int64_t gk = k0 + kk, gc = col0 + cv;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (gk < Kdim && gc < ldb) v = __ldg(reinterpret_cast<const uint4*>(B + gk * ldb + gc));
      *reinterpret_cast<uint4*>(&Bs[kk][cv]) = v;
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < kTK; ++kk) {
      const uint4 bv = *reinterpret_cast<const uint4*>(&Bs[kk][lane * 8]);
      float b[8];
      b[0] = __uint_as_float(bv.x << 16); b[1] = __uint_as_float(bv.x & 0xFFFF0000u);
      b[2] = __uint_as_float(bv.y << 16); b[3] = __uint_as_float(bv.y & 0xFFFF0000u);
      b[4] = __uint_as_float(bv.z << 16); b[5] = __uint_as_float(bv.z & 0xFFFF0000u);
      b[6] = __uint_as_float(bv.w << 16); b[7] = __uint_as_float(bv.w & 0xFFFF0000u);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float a = As[kk][warp * 4 + i];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a, b[j], acc[i][j]);
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t row = row0 + warp * 4 + i;          // warp-uniform
    if (row < Mdim) epi(row, col0 + lane * 8, acc[i]);
  }
}

// Epilogue of the projection: Adam on the low-rank state, bf16 direction to the workspace.
struct AdamEpilogue {
  StepScalars sc;
  float* M; float* V; int64_t ldmv;
  uint16_t* Nb; int64_t ldn;
  float* dbgR; float* dbgN; uint16_t* dbgNb;
  int64_t n;
  __device__ void operator()(int64_t i, int64_t j0, const float r8[8]) const {
    const int nvalid = (int)max((int64_t)0, min((int64_t)8, n - j0));
    if (nvalid == 0) return;
    float n8[8];
    adam8(sc, r8, M + i * ldmv + j0, V + i * ldmv + j0, nvalid, n8);
    if (nvalid == 8) {
      *reinterpret_cast<uint4*>(Nb + i * ldn + j0) = pack_bf16x8(n8);
    } else {
      for (int t = 0; t < nvalid; ++t) Nb[i * ldn + j0 + t] = float_to_bf16_bits(n8[t]);
    }
    if (dbgR) for (int t = 0; t < nvalid; ++t) dbgR[i * ldmv + j0 + t] = r8[t];
    if (dbgN) for (int t = 0; t < nvalid; ++t) dbgN[i * ldmv + j0 + t] = n8[t];
    if (dbgNb) for (int t = 0; t < nvalid; ++t) dbgNb[i * ldmv + j0 + t] = float_to_bf16_bits(n8[t]);
  }
};

// Epilogue of the back-projection: W' = dequant(W) - lr*alpha*D - lr*wd*dequant(W), then
// Quant_8 with stochastic rounding of the row's group (one warp = one group).
struct RequantEpilogue {
  StepScalars sc;
  qg_qtensor W;
  int ngroups;
  float* dbgW;
  __device__ void operator()(int64_t i, int64_t j0, const float d8[8]) const {
    const int nvalid = (int)max((int64_t)0, min((int64_t)8, W.cols - j0));
    const int g = (int)(j0 / kGroup);
    int8_t* codes = (int8_t*)W.codes + i * W.ld + j0;
    const float s = W.scales[i * ngroups + g], z = W.zeros[i * ngroups + g];
    float q[8], w[8];
    if (nvalid == 8) {
      unpack_int8x8(*reinterpret_cast<const uint2*>(codes), q);
    } else {
#pragma unroll
      for (int t = 0; t < 8; ++t) q[t] = (t < nvalid) ? (float)codes[t] : 0.f;
    }
    float mn = INFINITY, mx = -INFINITY;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      const float wh = __fmul_rn(__fsub_rn(q[t], z), s);
      w[t] = fmaf(-sc.lr_alpha, d8[t], fmaf(-sc.lr_wd, wh, wh));
      if (t < nvalid) { mn = fminf(mn, w[t]); mx = fmaxf(mx, w[t]); }
    }
    __syncwarp();
    mn = warp_min(mn);
    mx = warp_max(mx);
    const GroupParams gp = group_params<8>(mn, mx);
    if ((threadIdx.x & 31) == 0) { W.scales[i * ngroups + g] = gp.s; W.zeros[i * ngroups + g] = gp.z; }
    if (nvalid == 0) return;
    float h[8], c[8];
    sr_lanes8(sc, (uint32_t)i, (uint32_t)(j0 >> 3), h);
#pragma unroll
    for (int t = 0; t < 8; ++t) c[t] = sc.rounding == QG_ROUND_NEAREST ? rtn_code<8>(w[t], gp) : sr_code(w[t], gp, h[t]);
    if (nvalid == 8) {
      *reinterpret_cast<uint2*>(codes) = pack_int8x8(c);
    } else {
      for (int t = 0; t < nvalid; ++t) codes[t] = (int8_t)(int)c[t];
    }
    if (dbgW) for (int t = 0; t < nvalid; ++t) dbgW[i * W.ld + j0 + t] = w[t];
  }
};

}  // namespace

int launch_dequant_p(const qg_qtensor& P, uint16_t* out, int64_t ld_out, cudaStream_t st) {
  const int64_t threads = P.rows * (P.cols / 8);
  dequant_p_bf16_kernel<<<(unsigned)ceil_div(threads, 256), 256, 0, st>>>(P, out, ld_out);
  QG_LAUNCH_CHECK();
  return QG_OK;
}

size_t simt_workspace_bytes(int64_t m, int64_t n, int64_t r) {
  const size_t pt = (size_t)round_up(m * r * 2, 256);
  const size_t nb = (size_t)round_up(r * round_up(n, 64) * 2, 256);
  return pt + nb;
}

int launch_project_step_simt(const StepArgs& a, cudaStream_t st) {
  uint16_t* Pt = (uint16_t*)a.ws;
  uint16_t* Nb = (uint16_t*)((char*)a.ws + round_up(a.m * a.r * 2, 256));
  const int64_t ldn = round_up(a.n, 64);
  {
    const int rc = launch_dequant_p(a.P, Pt, a.r, st);
    if (rc != QG_OK) return rc;
  }
  {
    AdamEpilogue epi{a.sc, a.M, a.V, a.ldmv, Nb, ldn, a.dbg.R, a.dbg.N, a.dbg.N_b, a.n};
    dim3 grid((unsigned)ceil_div(a.n, kTN), (unsigned)ceil_div(a.r, kTM));
    gemm_simt_kernel<true, AdamEpilogue><<<grid, 256, 0, st>>>(Pt, a.r, a.G, a.ldg, a.r, a.n, a.m, epi);
    QG_LAUNCH_CHECK();
  }
  {
    RequantEpilogue epi{a.sc, a.W, (int)ceil_div(a.n, kGroup), a.dbg.W_pre};
    dim3 grid((unsigned)ceil_div(a.n, kTN), (unsigned)ceil_div(a.m, kTM));
    gemm_simt_kernel<false, RequantEpilogue><<<grid, 256, 0, st>>>(Pt, a.r, Nb, ldn, a.m, a.n, a.r, epi);
    QG_LAUNCH_CHECK();
  }
  return QG_OK;
}

}  // namespace qg
