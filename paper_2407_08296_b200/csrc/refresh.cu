// Subspace refresh (Sec. 3.5: "obtain the projection matrix using SVD"; Sec. 3.3: INT4 storage).
//
// The top-r left singular vectors of the gradient G (m x n, bf16) are found without a full SVD:
// block subspace iteration on G G^T with a block of b = r + oversample columns, followed by a
// Rayleigh-Ritz step that rotates the converged block onto the singular vectors.
//
//   Q <- orth(Gaussian m x b)
//   repeat iters times:   Z = G^T Q  (n x b);   Y = G Z  (m x b);   Q <- orth(Y)
//   Z = G^T Q;   T = Z^T Z  (b x b, summed in fp64);   T = X diag(lambda) X^T;   P = Q X[:, top r]
//
// The products with G run on the tensor cores (refresh_tc.cu: the fp32 iterate split into three bfloat16 planes,
// every product exact, fp32 accumulation); everything else is a generic fp32 GEMM kernel on the CUDA cores (fp64
// accumulation for T).  orth() is block Gram-Schmidt over panels of 64 columns with Cholesky QR of the panel: every
// projection twice and two rounds of Cholesky QR in the last iterations, one of each before.  The eigenvectors of T
// come from a one-sided (Hestenes) Jacobi iteration (rows kept in fp32, every sum in fp64: the result is INT4 in the
// end) over blocks of eight rows held on the SM, all sweeps in one cooperative launch with a grid barrier between the
// rounds of the tournament of blocks.  Each column of P is then given the sign that makes its largest entry positive,
// and P is quantized to INT4 (Quant_4).
//
// Several matrices of one shape are refreshed together (a "batch", up to kMaxBatch): every launch carries a matrix
// index beside its tile index and reads its operands from small pointer tables passed by value, so the few
// thousand small launches and the grid barriers of the eigen-iteration (about 1200) are paid once per batch instead of
// once per matrix.
//
// The singular values next to the r-th one sit in the noise bulk of the gradient with relative gaps of 1e-4..1e-3,
// and resolving that subspace to 1e-2 rad needs fp32-faithful products: plain bf16 tensor-core products of the
// iterate do not get there, the three-plane split does.
#include <cmath>
#include <mutex>

#include "qg_common.cuh"

namespace qg {

// refresh_tc.cu: the tensor-core route of the two products with the gradient
size_t split_planes_bytes(int64_t K, int64_t N);
bool split_gemm_supported(const uint16_t* A, int64_t sa_m, int64_t sa_k, int64_t M, int64_t N, int64_t K);
int launch_split_gemm(const uint16_t* A, int64_t sa_m, int64_t sa_k, const float* B, int64_t ldb, float* D, int64_t ldd,
                      int64_t M, int64_t N, int64_t K, uint16_t* planes, int32_t* status, cudaStream_t st);

namespace {

constexpr int kCoopDevices = 64;
std::mutex g_coop_mutex;
cudaEvent_t g_coop_done[kCoopDevices] = {};   // completion of the last cooperative launch, per device ordinal

// Test aid: 0 keeps every product of the refresh on the CUDA cores.
int g_refresh_tc = 1;
// Test aid: 0 rotates the rows of the Rayleigh-Ritz matrix pair by pair through L2 for every shape.
int g_jacobi_blocks = 1;

constexpr int kPanel = 64;    // columns orthonormalised together
constexpr int kMaxSweeps = 32;
constexpr int64_t kJacobiBytes = 64ll << 20;   // Rayleigh-Ritz matrices rotated by one launch: half of L2
constexpr int kGT = 64;       // GEMM tile (square), 16 x 16 threads, 4 x 4 outputs each
constexpr int kGK = 16;

constexpr int kMaxBatch = 8;  // matrices refreshed together
// One pointer per matrix of a batch, passed to the kernels by value.
template <class T>
struct Ptrs {
  T* p[kMaxBatch];
};
template <class T, class U>
Ptrs<T> offset_ptrs(const Ptrs<U>& src, int nb, int64_t off) {
  Ptrs<T> out{};
  for (int i = 0; i < nb; ++i) out.p[i] = src.p[i] + off;
  return out;
}

__device__ __forceinline__ float ld_as_float(const uint16_t* p, int64_t i) { return bf16_bits_to_float(p[i]); }
__device__ __forceinline__ float ld_as_float(const float* p, int64_t i) { return p[i]; }

// C[M x N] = alpha * A * B + beta * C.  A(i, k) = A[i * sa_m + k * sa_k], B(k, j) = B[k * sb_k + j * sb_n],
// C(i, j) = C[i * ldc + j].  TA is uint16_t (bfloat16 bits) or float; ACC/TC float or double.
// The grid's z index is (matrix of the batch) * slices + (slice of K).  With more than one slice, slice z writes
// its bare partial sums to part + z * M * N (row-major M x N) instead of C: products with a small result and a
// long K (the Gram matrices and projection coefficients of the orthonormalisation) would otherwise keep a
// handful of SMs busy.
template <class TA, class ACC, class TC>
__global__ void __launch_bounds__(256)
gemm_kernel(const Ptrs<const TA> Ab, int64_t sa_m, int64_t sa_k, const Ptrs<const float> Bb, int64_t sb_k, int64_t sb_n,
            const Ptrs<TC> Cb, int64_t ldc, int M, int N, int K, ACC alpha, ACC beta, int k_slice, int slices,
            const Ptrs<ACC> partb) {
  const int mat = (int)blockIdx.z / slices, slice = (int)blockIdx.z % slices;
  const TA* __restrict__ A = Ab.p[mat];
  const float* __restrict__ B = Bb.p[mat];
  TC* __restrict__ C = Cb.p[mat];
  ACC* __restrict__ part = slices > 1 ? partb.p[mat] : nullptr;
  // two buffers per operand: the loads of the next K step are in flight (in registers) while this one is multiplied
  __shared__ __align__(16) float As[2][kGK][kGT + 4];
  __shared__ __align__(16) float Bs[2][kGK][kGT + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int64_t m0 = (int64_t)blockIdx.y * kGT, n0 = (int64_t)blockIdx.x * kGT;
  ACC acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = (ACC)0;
  const bool a_m_fast = (sa_m == 1), b_n_fast = (sb_n == 1);
  const int k_begin = slice * k_slice;
  if (slices > 1) K = min(K, k_begin + k_slice);
  float ra[4], rb[4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      int mm, kk;
      if (a_m_fast) { mm = tid & 63; kk = (tid >> 6) + 4 * e; } else { kk = tid & 15; mm = (tid >> 4) + 16 * e; }
      const int64_t gm = m0 + mm, gk = k0 + kk;
      ra[e] = (gm < M && gk < K) ? ld_as_float(A, gm * sa_m + gk * sa_k) : 0.f;
      int nn, kb;
      if (b_n_fast) { nn = tid & 63; kb = (tid >> 6) + 4 * e; } else { kb = tid & 15; nn = (tid >> 4) + 16 * e; }
      const int64_t gn = n0 + nn, gkb = k0 + kb;
      rb[e] = (gn < N && gkb < K) ? B[gkb * sb_k + gn * sb_n] : 0.f;
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      int mm, kk;
      if (a_m_fast) { mm = tid & 63; kk = (tid >> 6) + 4 * e; } else { kk = tid & 15; mm = (tid >> 4) + 16 * e; }
      As[buf][kk][mm] = ra[e];
      int nn, kb;
      if (b_n_fast) { nn = tid & 63; kb = (tid >> 6) + 4 * e; } else { kb = tid & 15; nn = (tid >> 4) + 16 * e; }
      Bs[buf][kb][nn] = rb[e];
    }
  };
  if (k_begin < K) { fetch(k_begin); stash(0); }
  __syncthreads();
  int buf = 0;
  for (int k0 = k_begin; k0 < K; k0 += kGK, buf ^= 1) {
    const bool more = k0 + kGK < K;
    if (more) fetch(k0 + kGK);
#pragma unroll
    for (int kk = 0; kk < kGK; ++kk) {
      const float4 a4 = *reinterpret_cast<const float4*>(&As[buf][kk][ty * 4]);
      const float4 b4 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * 4]);
      const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] += (ACC)a[i] * (ACC)b[j];
    }
    if (more) stash(buf ^ 1);      // nobody reads that buffer before the barrier below
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      if (part != nullptr) {
        part[((int64_t)slice * M + gm) * N + gn] = acc[i][j];
        continue;
      }
      TC* c = C + gm * ldc + gn;
      const ACC v = alpha * acc[i][j] + (beta != (ACC)0 ? beta * (ACC)(*c) : (ACC)0);
      *c = (TC)v;
    }
  }
}

// C = alpha * (sum of the slices' partial sums, in slice order) + beta * C
template <class ACC, class TC>
__global__ void __launch_bounds__(256)
gemm_reduce_kernel(const Ptrs<ACC> partb, int slices, const Ptrs<TC> Cb, int64_t ldc, int M, int N, ACC alpha, ACC beta) {
  const ACC* __restrict__ part = partb.p[blockIdx.y];
  TC* __restrict__ C = Cb.p[blockIdx.y];
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)M * N) return;
  ACC s = (ACC)0;
  for (int z = 0; z < slices; ++z) s += part[(int64_t)z * M * N + idx];
  TC* c = C + (idx / N) * ldc + idx % N;
  *c = (TC)(alpha * s + (beta != (ACC)0 ? beta * (ACC)(*c) : (ACC)0));
}

int refresh_sm_count() {
  static int sms = 0;
  if (sms == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) sms = v;
    else sms = 148;
  }
  return sms;
}

constexpr int kSplitTiles = 160;         // products with fewer output tiles than this split their K range
constexpr int kSplitMinK = 128;          // ... into slices no shorter than this
constexpr int64_t kSplitScratch = 32 << 20;  // bytes of partial sums a product may use

// One product per matrix of the batch.  `part` (kSplitScratch bytes per matrix, or null tables) lets a product
// with few output tiles and a long K run as slices.
template <class TA, class ACC, class TC>
int gemm(int nb, const Ptrs<const TA>& A, int64_t sa_m, int64_t sa_k, const Ptrs<const float>& B, int64_t sb_k, int64_t sb_n,
         const Ptrs<TC>& C, int64_t ldc, int64_t M, int64_t N, int64_t K, ACC alpha, ACC beta, cudaStream_t st,
         const Ptrs<void>* part = nullptr) {
  if (M <= 0 || N <= 0) return QG_OK;
  dim3 grid((unsigned)ceil_div(N, kGT), (unsigned)ceil_div(M, kGT));
  const int64_t tiles = (int64_t)grid.x * grid.y * nb;
  int64_t slices = 1;
  if (part != nullptr && tiles < kSplitTiles && K >= 2 * kSplitMinK) {
    slices = ceil_div(2 * (int64_t)refresh_sm_count(), tiles);
    if (slices > K / kSplitMinK) slices = K / kSplitMinK;
    const int64_t fit = kSplitScratch / (M * N * (int64_t)sizeof(ACC));
    if (slices > fit) slices = fit;
  }
  Ptrs<ACC> pt{};
  if (slices <= 1) {
    grid.z = (unsigned)nb;
    gemm_kernel<TA, ACC, TC><<<grid, 256, 0, st>>>(A, sa_m, sa_k, B, sb_k, sb_n, C, ldc, (int)M, (int)N, (int)K, alpha, beta,
                                                   (int)K, 1, pt);
    QG_LAUNCH_CHECK();
    return QG_OK;
  }
  for (int i = 0; i < nb; ++i) pt.p[i] = reinterpret_cast<ACC*>(part->p[i]);
  const int64_t k_slice = round_up(ceil_div(K, slices), kGK);
  const int nslices = (int)ceil_div(K, k_slice);
  grid.z = (unsigned)(nslices * nb);
  gemm_kernel<TA, ACC, TC><<<grid, 256, 0, st>>>(A, sa_m, sa_k, B, sb_k, sb_n, C, ldc, (int)M, (int)N, (int)K, alpha, beta,
                                                 (int)k_slice, nslices, pt);
  QG_LAUNCH_CHECK();
  gemm_reduce_kernel<ACC, TC><<<dim3((unsigned)ceil_div(M * N, 256), (unsigned)nb), 256, 0, st>>>(pt, nslices, C, ldc, (int)M, (int)N,
                                                                                                  alpha, beta);
  QG_LAUNCH_CHECK();
  return QG_OK;
}

// ---- Gaussian start block: Q[i][j] ~ N(0, 1) from Philox4x32-10 (counter (j / 4, i, 0, 0x51)) and Box-Muller
__global__ void __launch_bounds__(256)
gaussian_kernel(const Ptrs<float> Qb, int64_t ld, int64_t rows, int64_t cols, const Ptrs<const void> seeds) {
  float* __restrict__ Q = Qb.p[blockIdx.y];
  // the seed of matrix y travels in the pointer table's slot (a 64-bit value, not an address)
  const uint64_t seed = (uint64_t)reinterpret_cast<uintptr_t>(seeds.p[blockIdx.y]);
  const uint32_t seed_lo = (uint32_t)seed, seed_hi = (uint32_t)(seed >> 32);
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t quads = cols / 4;
  if (idx >= rows * quads) return;
  const int64_t i = idx / quads, jq = idx % quads;
  const uint4 x = philox4x32_10(make_uint4((uint32_t)jq, (uint32_t)i, 0u, 0x51u), make_uint2(seed_lo, seed_hi));
  const float u0 = ((float)x.x + 0.5f) * 2.3283064365386963e-10f, u1 = ((float)x.y + 0.5f) * 2.3283064365386963e-10f;
  const float u2 = ((float)x.z + 0.5f) * 2.3283064365386963e-10f, u3 = ((float)x.w + 0.5f) * 2.3283064365386963e-10f;
  const float r0 = sqrtf(-2.f * logf(u0)), r1 = sqrtf(-2.f * logf(u2));
  float s0, c0, s1, c1;
  sincospif(2.f * u1, &s0, &c0);
  sincospif(2.f * u3, &s1, &c1);
  *reinterpret_cast<float4*>(Q + i * ld + 4 * jq) = make_float4(r0 * c0, r0 * s0, r1 * c1, r1 * s1);
}

// ---- Cholesky factor of a 64 x 64 Gram matrix and the inverse of the factor, ONE WARP per matrix, binary32.
// S (row-major) = L L^T;  Linv = L^-1 (lower triangular, row-major).  A non-positive pivot raises
// QG_DEV_BAD_FACTOR and is replaced by a tiny positive number so that the run continues with finite values.
// The factorisation is a chain of 64 dependent steps whatever runs it, so it is laid out for the shortest step:
// lane r keeps rows r and r + 32 in registers, the pivot and the column under it travel by shuffles, every loop is
// unrolled (all register indices are constants), and nothing touches memory until L is complete.  The inverse is
// then taken column-wise (lane c owns columns c and c + 32) by forward substitution with L broadcast from shared
// memory.  Binary32 is enough here: S itself comes from a binary32 product, and where the basis has to be
// orthonormal to rounding the panel goes through this twice.
__global__ void __launch_bounds__(32)
chol64_inverse_kernel(const Ptrs<const float> Sb, const Ptrs<float> Linvb, int32_t* __restrict__ status) {
  static_assert(kPanel == 64, "two rows and two columns per lane");
  const float* __restrict__ S = Sb.p[blockIdx.x];
  float* __restrict__ Linv = Linvb.p[blockIdx.x];
  __shared__ float Ls[kPanel][kPanel + 1];
  __shared__ float rds[kPanel];                  // 1 / L[i][i]
  const int lane = threadIdx.x;
  float a0[32], a1[64];                          // row `lane` (its lower triangle ends at column 31) and row `lane + 32`
#pragma unroll
  for (int j = 0; j < 32; j += 4) {
    const float4 v = *reinterpret_cast<const float4*>(S + lane * kPanel + j);
    a0[j] = v.x; a0[j + 1] = v.y; a0[j + 2] = v.z; a0[j + 3] = v.w;
  }
#pragma unroll
  for (int j = 0; j < 64; j += 4) {
    const float4 v = *reinterpret_cast<const float4*>(S + (lane + 32) * kPanel + j);
    a1[j] = v.x; a1[j + 1] = v.y; a1[j + 2] = v.z; a1[j + 3] = v.w;
  }
  bool bad = false;
  // right-looking factorisation; entries right of a row's diagonal hold values that are never read
#pragma unroll
  for (int k = 0; k < kPanel; ++k) {
    float piv = __shfl_sync(0xFFFFFFFFu, k < 32 ? a0[k & 31] : a1[k], k & 31);
    if (!(piv > 0.f)) { bad = true; piv = 1e-30f; }
    float inv = rsqrtf(piv);
    inv = inv * fmaf(-0.5f * piv * inv, inv, 1.5f);        // one Newton step: the reciprocal root to rounding
    if (lane == (k & 31)) rds[k] = inv;
    float l0 = 0.f;
    if (k < 32) { l0 = (lane == k) ? piv * inv : a0[k & 31] * inv; a0[k & 31] = l0; }
    const float l1 = (k >= 32 && lane + 32 == k) ? piv * inv : a1[k] * inv;
    a1[k] = l1;
#pragma unroll
    for (int j = k + 1; j < kPanel; ++j) {
      const float ljk = __shfl_sync(0xFFFFFFFFu, j < 32 ? l0 : l1, j & 31);
      if (j < 32) a0[j & 31] = fmaf(-l0, ljk, a0[j & 31]);
      a1[j] = fmaf(-l1, ljk, a1[j]);
    }
  }
  if (bad && lane == 0 && status) atomicOr(status, QG_DEV_BAD_FACTOR);
#pragma unroll
  for (int j = 0; j < 32; ++j) Ls[lane][j] = a0[j];
#pragma unroll
  for (int j = 0; j < 64; ++j) Ls[lane + 32][j] = a1[j];
  __syncwarp();
  // X = L^-1, column c (rows c..63) in x0, column c + 32 (rows c + 32..63) in x1:
  // X[i][c] = ([i == c] - sum_{k < i} L[i][k] X[k][c]) / L[i][i], with X[k][c] = 0 above the diagonal
  float x0[64], x1[32];
#pragma unroll
  for (int i = 0; i < kPanel; ++i) {
    float s0 = (i == lane) ? 1.f : 0.f, s0b = 0.f, s1 = (i == lane + 32) ? 1.f : 0.f, s1b = 0.f;
#pragma unroll
    for (int k = 0; k < i; ++k) {
      const float lik = Ls[i][k];
      if (k & 1) s0b = fmaf(-lik, x0[k], s0b); else s0 = fmaf(-lik, x0[k], s0);
      if (k >= 32) { if (k & 1) s1b = fmaf(-lik, x1[k - 32], s1b); else s1 = fmaf(-lik, x1[k - 32], s1); }
    }
    const float rd = rds[i];
    x0[i] = (i >= lane) ? (s0 + s0b) * rd : 0.f;
    if (i >= 32) x1[i - 32] = (i >= lane + 32) ? (s1 + s1b) * rd : 0.f;
  }
#pragma unroll
  for (int i = 0; i < kPanel; ++i) {
    Linv[i * kPanel + lane] = x0[i];
    Linv[i * kPanel + lane + 32] = i >= 32 ? x1[i - 32] : 0.f;
  }
}

// ---- one-sided (Hestenes) Jacobi on the rows of the symmetric b x b matrix T (binary32): rows are rotated in
// pairs until they are mutually orthogonal.  Then row j is lambda_j x_j^T (from T X = X Lambda), so the
// eigenvectors are the normalised rows and no second matrix has to follow the rotations.  Round `rnd` of a
// sweep pairs the b indices by the round-robin tournament schedule.
__device__ __forceinline__ void tournament_pair(int nitems, int rnd, int k, int& p, int& q) {
  const int mod = nitems - 1;
  if (k == 0) { p = nitems - 1; q = rnd % mod; }
  else { p = (rnd + k) % mod; q = (rnd - k + mod) % mod; }
  if (p > q) { const int t = p; p = q; q = t; }
}

// Barrier across the CTAs of a cooperative launch (all resident at once): one counter that only grows.  A CTA
// arrives with a release-add that returns nothing and then polls the counter itself with acquire loads until all
// gridDim.x arrivals of this generation are in: one trip to L2 to arrive and one to see the last arrival, no
// hand-over through a second word.  The wait is bounded; when it runs out the caller flags the status word and
// every CTA leaves.  `gen` counts the barriers this CTA has passed.
constexpr uint32_t kGridWaitPolls = 1u << 24;
__device__ __forceinline__ bool grid_barrier(unsigned int* count, unsigned int& gen) {
  __syncthreads();
  int ok = 1;
  ++gen;
  if (threadIdx.x == 0) {
    const unsigned int target = gen * gridDim.x;
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(count), "r"(1u) : "memory");
    uint32_t polls = 0;
    unsigned int seen;
    for (;;) {
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(count) : "memory");
      if (seen >= target) break;
      if (++polls >= kGridWaitPolls) { ok = 0; break; }
    }
  }
  return __syncthreads_and(ok) != 0;
}

// All sweeps of all matrices of a batch in one cooperative launch.  A team of 128 threads takes a pair of rows of
// one matrix, NE elements of each row per thread, kept in registers between the three inner products and the
// rotation; four teams per CTA move in step.  A grid barrier follows every round (the next round pairs the rows
// differently); a round covers that round's pairs of every matrix, so the barriers are shared by the batch.
// Rows move between SMs from round to round, so they are read and written through L2 (.cg).  The sweep's
// largest normalised inner product of matrix i is collected in off[i][sweep]; a matrix stops rotating after its
// first sweep whose value is <= tol, the launch ends when all have, and QG_DEV_NOT_CONVERGED is flagged if one
// never does.
constexpr int kTeam = 128, kTeamsPerCta = 4;
template <int NE>
__global__ void __launch_bounds__(kTeam * kTeamsPerCta, NE <= 16 ? 2 : 1)   // two CTAs per SM while the rows fit 64 registers
jacobi_sweeps_kernel(const Ptrs<float> Tb, int nb, int b, int sweeps, double tol, const Ptrs<unsigned long long> offb,
                     unsigned int* __restrict__ sync_words, int32_t* __restrict__ status) {
  __shared__ double red[kTeamsPerCta][3][kTeam / 32];
  __shared__ double s_worst[kTeamsPerCta][kMaxBatch];
  const int team = threadIdx.x / kTeam, tt = threadIdx.x % kTeam, tw = tt >> 5, lane = threadIdx.x & 31;
  const int pairs = b / 2, jobs = pairs * nb, batch = (int)gridDim.x * kTeamsPerCta;
  unsigned int gen = 0;
  uint32_t active = (1u << nb) - 1u;                // matrices still rotating
  for (int sw = 0; sw < sweeps && active != 0u; ++sw) {
    if (tt < kMaxBatch) s_worst[team][tt] = 0.0;
    for (int rnd = 0; rnd < b - 1; ++rnd) {
      for (int k0 = 0; k0 < jobs; k0 += batch) {
        const int k = k0 + (int)blockIdx.x * kTeamsPerCta + team;
        const int mat = k < jobs ? k / pairs : 0;
        const bool live = k < jobs && ((active >> mat) & 1u);
        int p = 0, q = 0;
        if (live) tournament_pair(b, rnd, k - mat * pairs, p, q);
        float* tp = Tb.p[mat] + (int64_t)p * b;
        float* tq = Tb.p[mat] + (int64_t)q * b;
        float x[NE], y[NE];
#pragma unroll
        for (int e = 0; e < NE; ++e) {
          const int i = tt + kTeam * e;
          const bool in = live && i < b;
          x[e] = in ? __ldcg(tp + i) : 0.f;
          y[e] = in ? __ldcg(tq + i) : 0.f;
        }
        // the thread's few products in binary32 (each exact to 2^-24 of itself), everything summed across
        // threads in binary64
        float af = 0.f, cf = 0.f, df = 0.f;
#pragma unroll
        for (int e = 0; e < NE; ++e) { af = fmaf(x[e], x[e], af); df = fmaf(y[e], y[e], df); cf = fmaf(x[e], y[e], cf); }
        double a = (double)af, c = (double)cf, d = (double)df;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
          d += __shfl_xor_sync(0xFFFFFFFFu, d, o);
          c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
        }
        __syncthreads();                               // the previous job has read `red`
        if (lane == 0) { red[team][0][tw] = a; red[team][1][tw] = d; red[team][2][tw] = c; }
        __syncthreads();
        a = red[team][0][0] + red[team][0][1] + red[team][0][2] + red[team][0][3];
        d = red[team][1][0] + red[team][1][1] + red[team][1][2] + red[team][1][3];
        c = red[team][2][0] + red[team][2][1] + red[team][2][2] + red[team][2][3];
        const double denom = sqrt(a * d);
        const double rel = denom > 0.0 ? fabs(c) / denom : 0.0;
        if (live && tt == 0) s_worst[team][mat] = fmax(s_worst[team][mat], rel);
        if (live && rel >= 1e-9) {
          const double zeta = (d - a) / (2.0 * c);
          const double tn = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
          const double csd = 1.0 / sqrt(1.0 + tn * tn);
          const float cs = (float)csd, sn = (float)(csd * tn);
#pragma unroll
          for (int e = 0; e < NE; ++e) {
            const int i = tt + kTeam * e;
            if (i < b) {
              __stcg(tp + i, fmaf(cs, x[e], -sn * y[e]));
              __stcg(tq + i, fmaf(sn, x[e], cs * y[e]));
            }
          }
        }
      }
      if (rnd == b - 2) {
        __syncthreads();
        // only ever compared, so the monotone integer view of a non-negative double serves atomicMax
        if (tt < nb && s_worst[team][tt] > 0.0)
          atomicMax(offb.p[tt] + sw, (unsigned long long)__double_as_longlong(s_worst[team][tt]));
      }
      if (!grid_barrier(sync_words, gen)) {
        if (threadIdx.x == 0 && status) atomicOr(status, QG_DEV_WAIT_EXPIRED);
        return;
      }
    }
    for (int i = 0; i < nb; ++i)
      if (((active >> i) & 1u) && __longlong_as_double((long long)__ldcg(offb.p[i] + sw)) <= tol) active &= ~(1u << i);
    __syncthreads();                                 // s_worst is cleared at the top of the next sweep
  }
  if (active != 0u && blockIdx.x == 0 && threadIdx.x == 0 && status) atomicOr(status, QG_DEV_NOT_CONVERGED);
}

template <int NE>
int launch_jacobi(const Ptrs<float>& T, int nb, int64_t b, int sweeps, double tol, const Ptrs<unsigned long long>& off,
                  unsigned int* sync_words, int32_t* status, cudaStream_t st) {
  // one cooperative launch, never more CTAs than are resident at once
  int per_sm = 0;
  QG_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, jacobi_sweeps_kernel<NE>, kTeam * kTeamsPerCta, 0));
  const int64_t resident = (int64_t)per_sm * refresh_sm_count();
  if (resident < 1) { note_cuda_error(cudaErrorCooperativeLaunchTooLarge, "jacobi_sweeps_kernel occupancy"); return QG_CUDA_ERROR; }
  int64_t grid = ceil_div(b / 2 * nb, kTeamsPerCta);
  if (grid > resident) grid = resident;
  int bi = (int)b;
  Ptrs<float> Tc = T;
  Ptrs<unsigned long long> offc = off;
  void* args[] = {&Tc, &nb, &bi, &sweeps, &tol, &offc, &sync_words, &status};
  QG_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)jacobi_sweeps_kernel<NE>, dim3((unsigned)grid), dim3(kTeam * kTeamsPerCta),
                                          args, 0, st));
  count_launch();
  return QG_OK;
}

// ---- the same iteration with the rows in blocks of eight.  A sweep first rotates the pairs INSIDE every block
// (seven short rounds through L2, as above), then runs a round-robin tournament over the blocks: a CTA takes a pair
// of blocks (I, J), every team of 64 threads keeps one row of I in registers, the rows of J sit in shared memory,
// and eight inner rounds rotate every row of I against every row of J.  A row pair thus moves through L2 once per
// eight rotations and a grid barrier separates b/8 - 1 rounds instead of b - 1: rounds of the plain form move every
// matrix of the batch through L2 once per rotation and are bound by exactly that.
constexpr int kBlkRows = 8, kBlkTeam = 64, kBlkThreads = kBlkRows * kBlkTeam;

// A thread of a team holds NE elements of a row in groups of four consecutive ones: group g covers elements
// 256 g + 4 tt .. + 3 (tt = its index in the team of 64), so rows move as 16-byte pieces everywhere.
__device__ __forceinline__ int blk_elem(int g, int tt) { return 256 * g + 4 * tt; }

__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// One rotation of the rows x, y (NE elements each per thread) held by a team; all teams of the CTA call it together.
// Returns the normalised inner product the pair had; `rotated` tells whether x and y changed.
template <int NE>
__device__ __forceinline__ double team_rotate(float (&x)[NE], float (&y)[NE], bool live, double (*red)[2], int team, int tw,
                                              int lane, bool& rotated) {
  // the thread's few products in binary32 (each exact to 2^-24 of itself), everything summed across threads in
  // binary64
  float af = 0.f, cf = 0.f, df = 0.f;
#pragma unroll
  for (int e = 0; e < NE; ++e) { af = fmaf(x[e], x[e], af); df = fmaf(y[e], y[e], df); cf = fmaf(x[e], y[e], cf); }
  double a = (double)af, c = (double)cf, d = (double)df;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
    d += __shfl_xor_sync(0xFFFFFFFFu, d, o);
    c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
  }
  if (lane == 0) { red[0][tw] = a; red[1][tw] = d; red[2][tw] = c; }
  // only the two warps of the team meet here (named barrier 1 + team): the teams of a CTA drift apart within a
  // round, so that one team's loads and multiplications overlap another's reductions
  asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "r"(kBlkTeam) : "memory");
  a = red[0][0] + red[0][1];
  d = red[1][0] + red[1][1];
  c = red[2][0] + red[2][1];
  // The sums are binary64; the angle is formed from them in binary32 (the difference d - a first, in binary64):
  // the rows it turns are binary32, and the six dependent divisions and roots of the binary64 form were a third
  // of a rotation's time.
  const double ad = a * d;
  const float rel_f = ad > 0.0 ? fabsf((float)c) * rsqrtf((float)a) * rsqrtf((float)d) : 0.f;
  const double rel = (double)rel_f;
  rotated = live && rel_f >= 1e-9f;
  if (rotated) {
    const float zeta = __fdividef((float)(d - a), 2.0f * (float)c);
    const float az = fabsf(zeta);
    // tan = sign(zeta) / (|zeta| + sqrt(1 + zeta^2)); for |zeta| beyond 2^60 the square overflows and tan = 1 / (2 zeta)
    const float tn = az < 1.0e18f ? copysignf(__fdividef(1.0f, az + sqrtf(fmaf(zeta, zeta, 1.0f))), zeta) : __fdividef(0.5f, zeta);
    const float cs = rsqrtf(fmaf(tn, tn, 1.0f)), sn = cs * tn;
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      const float xn = fmaf(cs, x[e], -sn * y[e]);
      y[e] = fmaf(sn, x[e], cs * y[e]);
      x[e] = xn;
    }
  }
  return live ? rel : 0.0;
}

template <int NE>
__global__ void __launch_bounds__(kBlkThreads, NE <= 16 ? 2 : 1)
jacobi_block_kernel(const Ptrs<float> Tb, int nb, int b, int sweeps, double tol, const Ptrs<unsigned long long> offb,
                    unsigned int* __restrict__ sync_words, int32_t* __restrict__ status) {
  // three sets of eight rows of b floats: the rows of block J of this job and of the next one (the copy engine brings
  // the next job's rows in while this one rotates), and the rows of block I of the next job
  extern __shared__ __align__(16) float blk_smem[];
  __shared__ double red[kBlkRows][3][2];
  __shared__ double s_worst[kBlkRows][kMaxBatch];
  const int team = threadIdx.x / kBlkTeam, tt = threadIdx.x % kBlkTeam, tw = tt >> 5, lane = threadIdx.x & 31;
  const int nblk = b / kBlkRows, half = nblk / 2;
  const int cta_jobs = nb * half;                    // block pairs per outer round; also eight within-block pairs each
  const int set = kBlkRows * b;
  float* const rows_i_next = blk_smem + 2 * set;
  unsigned int gen = 0;
  uint32_t active = (1u << nb) - 1u;                 // matrices still rotating
  for (int sw = 0; sw < sweeps && active != 0u; ++sw) {
    if (tt < kMaxBatch) s_worst[team][tt] = 0.0;
    __syncthreads();
    // ---- the pairs inside every block: round `rnd` of the tournament of its eight rows, four pairs per block
    for (int rnd = 0; rnd < kBlkRows - 1; ++rnd) {
      for (int j0 = 0; j0 < cta_jobs; j0 += (int)gridDim.x) {
        const int k = (j0 + (int)blockIdx.x) * kBlkRows + team;     // pair index: (matrix, block, pair of the round)
        const int per_mat = nblk * (kBlkRows / 2);
        const bool in_range = j0 + (int)blockIdx.x < cta_jobs;
        const int mat = in_range ? k / per_mat : 0;
        const bool live = in_range && ((active >> mat) & 1u);
        int p = 0, q = 0;
        if (live) {
          const int rem = k - mat * per_mat;
          tournament_pair(kBlkRows, rnd, rem % (kBlkRows / 2), p, q);
          p += (rem / (kBlkRows / 2)) * kBlkRows;
          q += (rem / (kBlkRows / 2)) * kBlkRows;
        }
        float* tp = Tb.p[mat] + (int64_t)p * b;
        float* tq = Tb.p[mat] + (int64_t)q * b;
        float x[NE], y[NE];
#pragma unroll
        for (int g = 0; g < NE / 4; ++g) {
          const int i = blk_elem(g, tt);
          const bool in = live && i < b;
          const float4 vx = in ? __ldcg(reinterpret_cast<const float4*>(tp + i)) : make_float4(0.f, 0.f, 0.f, 0.f);
          const float4 vy = in ? __ldcg(reinterpret_cast<const float4*>(tq + i)) : make_float4(0.f, 0.f, 0.f, 0.f);
          x[4 * g] = vx.x; x[4 * g + 1] = vx.y; x[4 * g + 2] = vx.z; x[4 * g + 3] = vx.w;
          y[4 * g] = vy.x; y[4 * g + 1] = vy.y; y[4 * g + 2] = vy.z; y[4 * g + 3] = vy.w;
        }
        bool rotated;
        const double rel = team_rotate<NE>(x, y, live, red[team], team, tw, lane, rotated);
        if (live && tt == 0) s_worst[team][mat] = fmax(s_worst[team][mat], rel);
        if (rotated) {
#pragma unroll
          for (int g = 0; g < NE / 4; ++g) {
            const int i = blk_elem(g, tt);
            if (i < b) {
              __stcg(reinterpret_cast<float4*>(tp + i), make_float4(x[4 * g], x[4 * g + 1], x[4 * g + 2], x[4 * g + 3]));
              __stcg(reinterpret_cast<float4*>(tq + i), make_float4(y[4 * g], y[4 * g + 1], y[4 * g + 2], y[4 * g + 3]));
            }
          }
        }
        __syncthreads();                               // `red` is free again
      }
      if (!grid_barrier(sync_words, gen)) {
        if (threadIdx.x == 0 && status) atomicOr(status, QG_DEV_WAIT_EXPIRED);
        return;
      }
    }
    // ---- the pairs between blocks: round `orr` of the tournament of the blocks
    for (int orr = 0; orr < nblk - 1; ++orr) {
      // the jobs of this CTA in this round whose matrix still rotates, in order; `fetch` starts the copies of a job's
      // sixteen rows (the team's row of block I into rows_i_next, its row of block J into set `buf`)
      auto next_job = [&](int job) {
        while (job < cta_jobs && !((active >> (job / half)) & 1u)) job += (int)gridDim.x;
        return job;
      };
      auto rows_of = [&](int job, float*& ti, float*& tj) {
        const int mat = job / half;
        int bi = 0, bj = 0;
        tournament_pair(nblk, orr, job - mat * half, bi, bj);
        ti = Tb.p[mat] + ((int64_t)bi * kBlkRows + team) * b;   // this team's row of block I
        tj = Tb.p[mat] + ((int64_t)bj * kBlkRows + team) * b;   // the row of block J it brings in and takes out
      };
      auto fetch = [&](int job, int buf) {
        float *ti, *tj;
        rows_of(job, ti, tj);
#pragma unroll
        for (int g = 0; g < NE / 4; ++g) {
          const int i = blk_elem(g, tt);
          if (i < b) {
            cp_async_16(rows_i_next + team * b + i, ti + i);
            cp_async_16(blk_smem + buf * set + team * b + i, tj + i);
          }
        }
        cp_async_commit();
      };
      int job = next_job((int)blockIdx.x), buf = 0;
      if (job < cta_jobs) fetch(job, 0);
      while (job < cta_jobs) {
        const int mat = job / half;
        const int nxt = next_job(job + (int)gridDim.x);
        float *ti, *tj;
        rows_of(job, ti, tj);
        float* const rows_j = blk_smem + buf * set;
        cp_async_wait_all();
        float x[NE], y[NE];
        // the thread's own pieces of its row of block I: the very bytes its own copies wrote
#pragma unroll
        for (int g = 0; g < NE / 4; ++g) {
          const int i = blk_elem(g, tt);
          const float4 v = i < b ? *reinterpret_cast<const float4*>(rows_i_next + team * b + i) : make_float4(0.f, 0.f, 0.f, 0.f);
          x[4 * g] = v.x; x[4 * g + 1] = v.y; x[4 * g + 2] = v.z; x[4 * g + 3] = v.w;
        }
        __syncthreads();                               // every team's row of block J has landed
        if (nxt < cta_jobs) fetch(nxt, buf ^ 1);       // rows of the same round: nobody writes them before their job
        double worst = 0.0;
#pragma unroll 1
        for (int sft = 0; sft < kBlkRows; ++sft) {
          float* yr = rows_j + ((team + sft) & (kBlkRows - 1)) * b;
#pragma unroll
          for (int g = 0; g < NE / 4; ++g) {
            const int i = blk_elem(g, tt);
            const float4 v = i < b ? *reinterpret_cast<const float4*>(yr + i) : make_float4(0.f, 0.f, 0.f, 0.f);
            y[4 * g] = v.x; y[4 * g + 1] = v.y; y[4 * g + 2] = v.z; y[4 * g + 3] = v.w;
          }
          bool rotated;
          worst = fmax(worst, team_rotate<NE>(x, y, true, red[team], team, tw, lane, rotated));
          if (rotated) {
#pragma unroll
            for (int g = 0; g < NE / 4; ++g) {
              const int i = blk_elem(g, tt);
              if (i < b) *reinterpret_cast<float4*>(yr + i) = make_float4(y[4 * g], y[4 * g + 1], y[4 * g + 2], y[4 * g + 3]);
            }
          }
          __syncthreads();                             // the next round reads another team's row; `red` is free
        }
        if (tt == 0) s_worst[team][mat] = fmax(s_worst[team][mat], worst);
#pragma unroll
        for (int g = 0; g < NE / 4; ++g) {
          const int i = blk_elem(g, tt);
          if (i < b) {
            __stcg(reinterpret_cast<float4*>(ti + i), make_float4(x[4 * g], x[4 * g + 1], x[4 * g + 2], x[4 * g + 3]));
            __stcg(reinterpret_cast<float4*>(tj + i), *reinterpret_cast<const float4*>(rows_j + team * b + i));
          }
        }
        __syncthreads();                               // set `buf` may be refilled by the job after next
        job = nxt;
        buf ^= 1;
      }
      if (orr == nblk - 2) {
        __syncthreads();
        // only ever compared, so the monotone integer view of a non-negative double serves atomicMax
        if (tt < nb && s_worst[team][tt] > 0.0)
          atomicMax(offb.p[tt] + sw, (unsigned long long)__double_as_longlong(s_worst[team][tt]));
      }
      if (!grid_barrier(sync_words, gen)) {
        if (threadIdx.x == 0 && status) atomicOr(status, QG_DEV_WAIT_EXPIRED);
        return;
      }
    }
    for (int i = 0; i < nb; ++i)
      if (((active >> i) & 1u) && __longlong_as_double((long long)__ldcg(offb.p[i] + sw)) <= tol) active &= ~(1u << i);
    __syncthreads();                                 // s_worst is cleared at the top of the next sweep
  }
  if (active != 0u && blockIdx.x == 0 && threadIdx.x == 0 && status) atomicOr(status, QG_DEV_NOT_CONVERGED);
}

// Opts the instance into its dynamic shared memory once per device.
template <int NE>
int launch_jacobi_block(const Ptrs<float>& T, int nb, int64_t b, int sweeps, double tol, const Ptrs<unsigned long long>& off,
                        unsigned int* sync_words, int32_t* status, cudaStream_t st) {
  const int smem = (int)(3 * kBlkRows * b * sizeof(float));
  static bool smem_set[kCoopDevices] = {};
  int dev = 0;
  QG_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kCoopDevices) return QG_UNSUPPORTED_SHAPE;
  if (!smem_set[dev]) {
    QG_CUDA_TRY(cudaFuncSetAttribute(jacobi_block_kernel<NE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 3 * kBlkRows * NE * kBlkTeam * 4));
    smem_set[dev] = true;
  }
  // one cooperative launch, never more CTAs than are resident at once
  int per_sm = 0;
  QG_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, jacobi_block_kernel<NE>, kBlkThreads, smem));
  const int64_t resident = (int64_t)per_sm * refresh_sm_count();
  if (resident < 1) { note_cuda_error(cudaErrorCooperativeLaunchTooLarge, "jacobi_block_kernel occupancy"); return QG_CUDA_ERROR; }
  int64_t grid = (b / kBlkRows / 2) * nb;
  if (grid > resident) grid = resident;
  int bi = (int)b;
  Ptrs<float> Tc = T;
  Ptrs<unsigned long long> offc = off;
  void* args[] = {&Tc, &nb, &bi, &sweeps, &tol, &offc, &sync_words, &status};
  QG_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)jacobi_block_kernel<NE>, dim3((unsigned)grid), dim3(kBlkThreads), args,
                                          (size_t)smem, st));
  count_launch();
  return QG_OK;
}

// lambda_j = norm of row j of the rotated T (= |eigenvalue j|); rank_j = its position in descending order
__global__ void __launch_bounds__(128)
row_norm_kernel(const Ptrs<const float> Tb, int b, const Ptrs<double> lamb) {
  const float* row = Tb.p[blockIdx.y] + (int64_t)blockIdx.x * b;
  double* __restrict__ lam = lamb.p[blockIdx.y];
  double s = 0.0;
  for (int i = threadIdx.x; i < b; i += blockDim.x) s += (double)row[i] * (double)row[i];
  __shared__ double red[4];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) lam[blockIdx.x] = sqrt(red[0] + red[1] + red[2] + red[3]);
}

// Xsel[i][rank_j] = X[i][j] = T[j][i] / lambda_j for the r largest lambda_j
__global__ void __launch_bounds__(256)
select_top_kernel(const Ptrs<const float> Tb, const Ptrs<const double> lamb, int b, int r, const Ptrs<float> Xselb) {
  const float* __restrict__ T = Tb.p[blockIdx.y];
  const double* __restrict__ lam = lamb.p[blockIdx.y];
  float* __restrict__ Xsel = Xselb.p[blockIdx.y];
  const int j = blockIdx.x;
  const double lj = lam[j];
  __shared__ int s_rank;
  if (threadIdx.x == 0) s_rank = 0;
  __syncthreads();
  int cnt = 0;
  for (int k = threadIdx.x; k < b; k += blockDim.x) {
    const double lk = lam[k];
    cnt += (lk > lj || (lk == lj && k < j)) ? 1 : 0;
  }
  atomicAdd(&s_rank, cnt);
  __syncthreads();
  const int rank = s_rank;
  if (rank >= r) return;
  const double inv = lj > 0.0 ? 1.0 / lj : 0.0;
  for (int i = threadIdx.x; i < b; i += blockDim.x) Xsel[(int64_t)i * r + rank] = (float)((double)T[(int64_t)j * b + i] * inv);
}

// Each column of P gets the sign that makes its largest-magnitude entry positive; optional copy to P_out.
__global__ void __launch_bounds__(256)
sign_fix_kernel(const Ptrs<float> Pb, int64_t m, int r, const Ptrs<float> P_outb) {
  float* __restrict__ P = Pb.p[blockIdx.y];
  float* __restrict__ P_out = P_outb.p[blockIdx.y];
  const int j = blockIdx.x;
  float best = 0.f, bestv = 0.f;
  for (int64_t i = threadIdx.x; i < m; i += blockDim.x) {
    const float v = P[i * r + j];
    if (fabsf(v) > best) { best = fabsf(v); bestv = v; }
  }
  __shared__ float sb[256], sv[256];
  sb[threadIdx.x] = best; sv[threadIdx.x] = bestv;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o && sb[threadIdx.x + o] > sb[threadIdx.x]) { sb[threadIdx.x] = sb[threadIdx.x + o]; sv[threadIdx.x] = sv[threadIdx.x + o]; }
    __syncthreads();
  }
  const float sgn = sv[0] < 0.f ? -1.f : 1.f;
  for (int64_t i = threadIdx.x; i < m; i += blockDim.x) {
    const float v = P[i * r + j] * sgn;
    P[i * r + j] = v;
    if (P_out) P_out[i * r + j] = v;
  }
}

struct RefreshWs {
  float *Q, *Y, *Z, *Wp, *Cb, *S, *Linv, *Xsel, *P32;
  void* part;      // partial sums of sliced products
  uint16_t* planes;  // the three bfloat16 planes of an iterate, for the tensor-core products
  float* T;        // the Rayleigh-Ritz matrix, then its rotated rows
  double *lam, *off;
  int32_t* done;
};

size_t carve_refresh(void* base, int64_t m, int64_t n, int64_t b, int64_t r, RefreshWs* w) {
  size_t off = 0;
  auto take = [&](size_t bytes) { void* p = base ? (char*)base + off : nullptr; off += (size_t)round_up((int64_t)bytes, 256); return p; };
  RefreshWs t{};
  t.T = (float*)take((size_t)b * b * 4);
  t.lam = (double*)take((size_t)b * 8);
  t.off = (double*)take(kMaxSweeps * 8);     // largest normalised inner product of each sweep
  t.done = (int32_t*)take(8);               // the two words of the grid barrier
  t.Q = (float*)take((size_t)m * b * 4);
  t.Y = (float*)take((size_t)m * b * 4);
  t.Z = (float*)take((size_t)n * b * 4);
  t.Wp = (float*)take((size_t)m * kPanel * 4);
  t.Cb = (float*)take((size_t)b * kPanel * 4);
  t.S = (float*)take((size_t)kPanel * kPanel * 4);
  t.Linv = (float*)take((size_t)kPanel * kPanel * 4);
  t.Xsel = (float*)take((size_t)b * r * 4);
  t.P32 = (float*)take((size_t)m * r * 4);
  t.part = take((size_t)kSplitScratch);
  t.planes = (uint16_t*)take(split_planes_bytes(m > n ? m : n, b));
  if (w) *w = t;
  return off;
}

// The workspaces of the matrices of one batch, and pointer tables into them.
struct Batch {
  int nb;
  RefreshWs w[kMaxBatch];
  template <class T, class F>
  Ptrs<T> tab(F field, int64_t off = 0) const {
    Ptrs<T> t{};
    for (int i = 0; i < nb; ++i) t.p[i] = field(w[i]) + off;
    return t;
  }
};
#define QG_TAB(T, member) bt.tab<T>([](const RefreshWs& x) { return x.member; })
#define QG_TAB_OFF(T, member, off) bt.tab<T>([](const RefreshWs& x) { return x.member; }, (off))

// Q <- orthonormal basis of the columns of Y (m x b, both pitch b), panel by panel, for every matrix of the batch.
// `full`: every projection applied twice and two rounds of Cholesky QR per panel: orthonormal to fp32 rounding, what
// the Rayleigh-Ritz step and the returned vectors need.  Otherwise one of each: the basis comes out orthonormal to
// about 1e-2 (fp32 Gram matrices of panels with a condition number of several hundred), which is all an
// intermediate subspace iteration asks of it: the next multiplication by G G^T and the next orthonormalisation
// start from that basis, they do not inherit its error.
int orthonormalize(const Batch& bt, int64_t m, int64_t b, int32_t* status, cudaStream_t st, bool full) {
  const int passes = full ? 2 : 1;
  const int nb = bt.nb;
  Ptrs<void> part{};
  for (int i = 0; i < nb; ++i) part.p[i] = bt.w[i].part;
  const Ptrs<const float> Q = QG_TAB(const float, Q);
  const Ptrs<float> Cb = QG_TAB(float, Cb), S = QG_TAB(float, S), Linv = QG_TAB(float, Linv), Wp = QG_TAB(float, Wp);
  const Ptrs<const float> Cbc = QG_TAB(const float, Cb), Sc = QG_TAB(const float, S), Linvc = QG_TAB(const float, Linv),
                          Wpc = QG_TAB(const float, Wp);
  for (int64_t j0 = 0; j0 < b; j0 += kPanel) {
    const Ptrs<float> Yj = QG_TAB_OFF(float, Y, j0), Qj = QG_TAB_OFF(float, Q, j0);
    const Ptrs<const float> Yjc = QG_TAB_OFF(const float, Y, j0);
    int rc;
    for (int pass = 0; pass < passes && j0 > 0; ++pass) {
      // C = Q[:, :j0]^T Yj   (j0 x 64);   Yj -= Q[:, :j0] C
      rc = gemm<float, float, float>(nb, Q, 1, b, Yjc, b, 1, Cb, kPanel, j0, kPanel, m, 1.f, 0.f, st, &part);
      if (rc != QG_OK) return rc;
      rc = gemm<float, float, float>(nb, Q, b, 1, Cbc, kPanel, 1, Yj, b, m, kPanel, j0, -1.f, 1.f, st, &part);
      if (rc != QG_OK) return rc;
    }
    // Cholesky QR on the panel, two rounds (Yj -> Wp -> Qj) or one (Yj -> Qj)
    for (int pass = 0; pass < passes; ++pass) {
      const bool last = pass + 1 == passes;
      const Ptrs<const float>& src = pass == 0 ? Yjc : Wpc;
      const int64_t lds = pass == 0 ? b : kPanel;
      const Ptrs<float>& dst = last ? Qj : Wp;
      const int64_t ldd = last ? b : kPanel;
      rc = gemm<float, float, float>(nb, src, 1, lds, src, lds, 1, S, kPanel, kPanel, kPanel, m, 1.f, 0.f, st, &part);
      if (rc != QG_OK) return rc;
      chol64_inverse_kernel<<<nb, 32, 0, st>>>(Sc, Linv, status);
      QG_LAUNCH_CHECK();
      // dst = src * Linv^T:  B(k, j) = Linv[j][k]
      rc = gemm<float, float, float>(nb, src, lds, 1, Linvc, 1, kPanel, dst, ldd, m, kPanel, kPanel, 1.f, 0.f, st);
      if (rc != QG_OK) return rc;
    }
  }
  return QG_OK;
}

}  // namespace

size_t refresh_workspace_bytes(int64_t m, int64_t n, int64_t b) { return carve_refresh(nullptr, m, n, b, b, nullptr); }

// One batch (at most kMaxBatch matrices of one shape).  `transposed`: the singular vectors wanted are the RIGHT ones
// of G, i.e. the left ones of G^T; G is then read with its two strides swapped and (m, n) are the extents of G^T.
static int refresh_batch(const RefreshJob* jobs, int nb, int64_t m, int64_t n, int64_t r, int64_t b, int iters, int sweeps,
                         char* ws, size_t ws_stride, int32_t* status, cudaStream_t st, bool transposed) {
  Batch bt{};
  bt.nb = nb;
  Ptrs<const uint16_t> G{};
  Ptrs<const void> seeds{};
  Ptrs<float> P_out{};
  int64_t ldg = jobs[0].ldg;
  for (int i = 0; i < nb; ++i) {
    carve_refresh(ws + (size_t)i * ws_stride, m, n, b, r, &bt.w[i]);
    G.p[i] = jobs[i].G;
    seeds.p[i] = reinterpret_cast<const void*>((uintptr_t)jobs[i].seed);
    P_out.p[i] = jobs[i].P_fp32;
    if (jobs[i].ldg != ldg) return QG_INVALID_ARGUMENT;          // one pitch per batch (the caller groups by it)
  }
  const int64_t rs = transposed ? 1 : ldg, cs = transposed ? ldg : 1;   // strides between rows / columns of the matrix
  const Ptrs<const float> Q = QG_TAB(const float, Q), Z = QG_TAB(const float, Z), Xsel = QG_TAB(const float, Xsel);
  const Ptrs<float> Y = QG_TAB(float, Y), Zw = QG_TAB(float, Z), P32 = QG_TAB(float, P32);
  int rc;
  // start block
  {
    const int64_t threads = m * (b / 4);
    gaussian_kernel<<<dim3((unsigned)ceil_div(threads, 256), (unsigned)nb), 256, 0, st>>>(Y, b, m, b, seeds);
    QG_LAUNCH_CHECK();
    rc = orthonormalize(bt, m, b, status, st, iters < 2);          // in full only if no later iteration will be
    if (rc != QG_OK) return rc;
  }
  // The two products with the gradient go to the tensor cores (bfloat16 gradient times an iterate split into three
  // bfloat16 planes, fp32 accumulation: refresh_tc.cu), one launch per matrix, where shape and strides allow it.
  // Their rounding differs from the CUDA-core kernel's only in the order of an fp32 accumulation; measured, the
  // largest principal angle to the exact subspace is the same to three digits either way (it is set by the number
  // of iterations, 5e-3 rad on the rectangular LLaMA shapes after 12, not by the arithmetic).  Only the product that
  // feeds the Rayleigh-Ritz step keeps the CUDA-core kernel, whose accumulation is not biased toward zero.
  const bool tc_z = g_refresh_tc && split_gemm_supported(G.p[0], cs, rs, n, b, m);   // Z = X^T Q: A(i, k) = X[k][i]
  const bool tc_y = g_refresh_tc && split_gemm_supported(G.p[0], rs, cs, m, b, n);   // Y = X Z:   A(i, k) = X[i][k]
  for (int it = 0; it <= iters; ++it) {
    // Z = G^T Q
    if (tc_z && it < iters) {
      for (int i = 0; i < nb; ++i) {
        rc = launch_split_gemm(G.p[i], cs, rs, bt.w[i].Q, b, bt.w[i].Z, b, n, b, m, bt.w[i].planes, status, st);
        if (rc != QG_OK) return rc;
      }
    } else {
      rc = gemm<uint16_t, float, float>(nb, G, cs, rs, Q, b, 1, Zw, b, n, b, m, 1.f, 0.f, st);
      if (rc != QG_OK) return rc;
    }
    if (it == iters) break;
    // Y = G Z
    if (tc_y) {
      for (int i = 0; i < nb; ++i) {
        rc = launch_split_gemm(G.p[i], rs, cs, bt.w[i].Z, b, bt.w[i].Y, b, m, b, n, bt.w[i].planes, status, st);
        if (rc != QG_OK) return rc;
      }
    } else {
      rc = gemm<uint16_t, float, float>(nb, G, rs, cs, Z, b, 1, Y, b, m, b, n, 1.f, 0.f, st);
      if (rc != QG_OK) return rc;
    }
    rc = orthonormalize(bt, m, b, status, st, it + 2 >= iters);   // the last two in full
    if (rc != QG_OK) return rc;
  }
  // Rayleigh-Ritz: T = Z^T Z (accumulated in binary64, kept in binary32), eigenvectors by one-sided Jacobi
  const Ptrs<float> T = QG_TAB(float, T);
  const Ptrs<double> lam = QG_TAB(double, lam);
  rc = gemm<float, double, float>(nb, Z, 1, b, Z, b, 1, T, b, b, b, n, 1.0, 0.0, st);
  if (rc != QG_OK) return rc;
  if (sweeps > kMaxSweeps) sweeps = kMaxSweeps;
  for (int i = 0; i < nb; ++i) QG_CUDA_TRY(cudaMemsetAsync(bt.w[i].off, 0, kMaxSweeps * 8, st));
  // A round of the row-by-row form reads and writes every row once, so the matrices rotated together should stay in
  // L2 together: at most kJacobiBytes of them per cooperative launch.
  const bool blocks = g_jacobi_blocks && b % (2 * kBlkRows) == 0 && b <= 32 * kBlkTeam;
  // (the block form moves a row through L2 once per eight rotations and takes the whole batch in one launch: more
  // jobs per round leave fewer CTAs idle at its end)
  const int per_launch = blocks ? nb : (int)std::max<int64_t>(1, std::min<int64_t>(nb, kJacobiBytes / (b * b * 4)));
  for (int first = 0; first < nb; first += per_launch) {
    const int cnt = std::min(per_launch, nb - first);
    Ptrs<float> Tsub{};
    Ptrs<unsigned long long> off{};
    for (int i = 0; i < cnt; ++i) {
      Tsub.p[i] = bt.w[first + i].T;
      off.p[i] = reinterpret_cast<unsigned long long*>(bt.w[first + i].off);
    }
    QG_CUDA_TRY(cudaMemsetAsync(bt.w[0].done, 0, 8, st));
    unsigned int* sync_words = reinterpret_cast<unsigned int*>(bt.w[0].done);
    // the iteration converges quadratically at the end: a sweep that met nothing above 1e-5 leaves ~1e-10
    constexpr double kTol = 1e-5;
    // Refreshes may run on several streams at once (their many small kernels overlap well), but two grids whose
    // CTAs wait for one another must never be half resident together: each cooperative launch waits for the
    // previous one of this process on the device, whatever its stream.
    std::lock_guard<std::mutex> lock(g_coop_mutex);
    int dev = 0;
    QG_CUDA_TRY(cudaGetDevice(&dev));
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    QG_CUDA_TRY(cudaStreamIsCapturing(st, &cap));
    const bool chain = cap == cudaStreamCaptureStatusNone && dev >= 0 && dev < kCoopDevices;
    if (chain) {
      if (!g_coop_done[dev]) QG_CUDA_TRY(cudaEventCreateWithFlags(&g_coop_done[dev], cudaEventDisableTiming));
      else QG_CUDA_TRY(cudaStreamWaitEvent(st, g_coop_done[dev], 0));
    }
    // rows in blocks of eight where the block count is even and a block fits shared memory; else row by row
    if (blocks && b <= 16 * kBlkTeam) rc = launch_jacobi_block<16>(Tsub, cnt, b, sweeps, kTol, off, sync_words, status, st);
    else if (blocks) rc = launch_jacobi_block<32>(Tsub, cnt, b, sweeps, kTol, off, sync_words, status, st);
    else if (b <= 8 * kTeam) rc = launch_jacobi<8>(Tsub, cnt, b, sweeps, kTol, off, sync_words, status, st);
    else if (b <= 16 * kTeam) rc = launch_jacobi<16>(Tsub, cnt, b, sweeps, kTol, off, sync_words, status, st);
    else rc = launch_jacobi<32>(Tsub, cnt, b, sweeps, kTol, off, sync_words, status, st);
    if (rc != QG_OK) return rc;
    if (chain) QG_CUDA_TRY(cudaEventRecord(g_coop_done[dev], st));
  }
  const Ptrs<const float> Tc = QG_TAB(const float, T);
  const Ptrs<const double> lamc = QG_TAB(const double, lam);
  row_norm_kernel<<<dim3((unsigned)b, (unsigned)nb), 128, 0, st>>>(Tc, (int)b, lam);
  QG_LAUNCH_CHECK();
  select_top_kernel<<<dim3((unsigned)b, (unsigned)nb), 256, 0, st>>>(Tc, lamc, (int)b, (int)r, QG_TAB(float, Xsel));
  QG_LAUNCH_CHECK();
  // P = Q Xsel
  rc = gemm<float, float, float>(nb, Q, b, 1, Xsel, r, 1, P32, r, m, r, b, 1.f, 0.f, st);
  if (rc != QG_OK) return rc;
  sign_fix_kernel<<<dim3((unsigned)r, (unsigned)nb), 256, 0, st>>>(P32, m, (int)r, P_out);
  QG_LAUNCH_CHECK();
  for (int i = 0; i < nb; ++i) {
    rc = launch_quantize_rtn(jobs[i].P_new->bits, bt.w[i].P32, m, r, r, jobs[i].P_new, st);
    if (rc != QG_OK) return rc;
  }
  return QG_OK;
}

// `count` matrices of one shape, in batches of as many as the workspace holds (at most kMaxBatch).
int launch_refresh_batched(const RefreshJob* jobs, int count, int64_t m, int64_t n, int64_t r, int64_t b, int iters, int sweeps,
                           void* ws, size_t ws_bytes, int32_t* status, cudaStream_t st, bool transposed) {
  const size_t stride = refresh_workspace_bytes(m, n, b);
  int64_t fit = (int64_t)(ws_bytes / stride);
  if (fit < 1) return QG_WORKSPACE_TOO_SMALL;
  if (fit > kMaxBatch) fit = kMaxBatch;
  for (int first = 0; first < count; first += (int)fit) {
    const int nb = count - first < (int)fit ? count - first : (int)fit;
    const int rc = refresh_batch(jobs + first, nb, m, n, r, b, iters, sweeps, reinterpret_cast<char*>(ws), stride, status, st,
                                 transposed);
    if (rc != QG_OK) return rc;
  }
  return QG_OK;
}

int set_refresh_tc(int on) { g_refresh_tc = on ? 1 : 0; return QG_OK; }
int set_jacobi_blocks(int on) { g_jacobi_blocks = on ? 1 : 0; return QG_OK; }

int launch_refresh(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r, int64_t b, int iters, int sweeps,
                   uint64_t seed, const qg_qtensor* P_new, float* P_fp32, void* ws, size_t ws_bytes, int32_t* status,
                   cudaStream_t st, bool transposed) {
  const RefreshJob job{G, ldg, seed, P_new, P_fp32};
  return launch_refresh_batched(&job, 1, m, n, r, b, iters, sweeps, ws, ws_bytes, status, st, transposed);
}

}  // namespace qg
