// extern "C" boundary of the Q-GaLore library: argument validation, scalar preparation and
// dispatch to the kernels.  Nothing here allocates or synchronises.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <vector>

#include "qg_common.cuh"

namespace qg {

static thread_local char g_last_error[256] = "";
static std::atomic<uint64_t> g_launches{0};

void note_cuda_error(cudaError_t e, const char* where) {
  snprintf(g_last_error, sizeof(g_last_error), "%s: %s (%s)", where, cudaGetErrorName(e), cudaGetErrorString(e));
  (void)cudaGetLastError();  // clear the sticky-less error so that later calls start clean
}
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int launch_project_step_simt(const StepArgs& a, cudaStream_t st);
size_t simt_workspace_bytes(int64_t m, int64_t n, int64_t r);
int launch_project_step_tc(const StepArgs& a, cudaStream_t st);
size_t tc_workspace_bytes(int64_t m, int64_t n, int64_t r);
int launch_refresh(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r, int64_t b, int iters, int sweeps,
                   uint64_t seed, const qg_qtensor* P_new, float* P_fp32, void* ws, size_t ws_bytes, int32_t* status,
                   cudaStream_t st, bool transposed);
size_t refresh_workspace_bytes(int64_t m, int64_t n, int64_t b);
int launch_refresh_batched(const RefreshJob* jobs, int count, int64_t m, int64_t n, int64_t r, int64_t b, int iters, int sweeps,
                           void* ws, size_t ws_bytes, int32_t* status, cudaStream_t st, bool transposed);
struct Plan;
size_t plan_table_bytes(const StepArgs* items, int32_t count);
int plan_create(const StepArgs* items, int32_t count, void* table_dev, size_t table_bytes, void* workspace,
                size_t workspace_bytes, Plan** out);
int plan_step(const Plan* plan, const StepScalars& sc, int32_t* status, cudaStream_t st, cudaEvent_t* ev);
int plan_step_timed(const Plan* plan, const StepScalars& sc, int32_t* status, cudaStream_t st, float* ms,
                    int32_t* launches);
void plan_destroy(Plan* plan);
int tc_kernel_info(char* buf, size_t cap);
int set_pair_mode(int mask);
int set_fused_dequant(int on);
int set_refresh_tc(int on);
int set_jacobi_blocks(int on);
int set_chunk_budget(size_t bytes);

static int g_step_impl = 0;  // 0: tensor-core kernels; 1: CUDA-core kernels (validation aid)

}  // namespace qg

using namespace qg;

extern "C" {

const char* qgalore_status_string(int status) {
  switch (status) {
    case QG_OK: return "ok";
    case QG_INVALID_ARGUMENT: return "invalid argument";
    case QG_UNSUPPORTED_SHAPE: return "unsupported shape";
    case QG_MISALIGNED: return "misaligned pointer or row pitch";
    case QG_WORKSPACE_TOO_SMALL: return "workspace too small";
    case QG_CUDA_ERROR: return "CUDA error";
    case QG_NOT_CONVERGED: return "not converged";
    default: return "unknown status";
  }
}

const char* qgalore_last_cuda_error(void) { return g_last_error; }
const char* qgalore_kernel_revision(void) { return QG_STEP_KERNELS_REVISION; }
uint64_t qgalore_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

static int quantize_common(int bits, const float* src, int64_t rows, int64_t cols, int64_t ld_src,
                           const qg_qtensor* dst, void* stream) {
  if (!src || rows <= 0 || cols <= 0 || ld_src < cols) return QG_INVALID_ARGUMENT;
  int rc = check_qtensor(dst, bits);
  if (rc != QG_OK) return rc;
  if (dst->rows != rows || dst->cols != cols) return QG_INVALID_ARGUMENT;
  if (!aligned16(src) || ld_src % 4 != 0) return QG_MISALIGNED;
  return launch_quantize_rtn(bits, src, rows, cols, ld_src, dst, (cudaStream_t)stream);
}

int qgalore_quantize_int4(const float* src, int64_t rows, int64_t cols, int64_t ld_src, const qg_qtensor* dst,
                          void* stream) {
  return quantize_common(4, src, rows, cols, ld_src, dst, stream);
}

int qgalore_quantize_int2(const float* src, int64_t rows, int64_t cols, int64_t ld_src, const qg_qtensor* dst,
                          void* stream) {
  return quantize_common(2, src, rows, cols, ld_src, dst, stream);
}

int qgalore_quantize_int8(const float* src, int64_t rows, int64_t cols, int64_t ld_src, const qg_qtensor* dst,
                          void* stream) {
  return quantize_common(8, src, rows, cols, ld_src, dst, stream);
}

int qgalore_dequantize(const qg_qtensor* src, float* dst, int64_t ld_dst, void* stream) {
  if (!src || !dst) return QG_INVALID_ARGUMENT;
  if (src->bits != 2 && src->bits != 4 && src->bits != 8) return QG_INVALID_ARGUMENT;
  int rc = check_qtensor(src, src->bits);
  if (rc != QG_OK) return rc;
  if (ld_dst < src->cols) return QG_INVALID_ARGUMENT;
  if (!aligned16(dst) || ld_dst % 4 != 0) return QG_MISALIGNED;
  return launch_dequantize(src, dst, ld_dst, (cudaStream_t)stream);
}

// --- App. A: the INT8 linear layer ------------------------------------------------------------
static int check_bf16_matrix(const uint16_t* p, int64_t rows, int64_t cols, int64_t ld) {
  if (!p || rows <= 0 || cols <= 0 || ld < cols) return QG_INVALID_ARGUMENT;
  if (!aligned16(p) || ld % 8 != 0) return QG_MISALIGNED;
  return QG_OK;
}
static bool linear_extent_ok(int64_t v) { return v > 0 && v <= (int64_t)1 << 30; }

int qgalore_int8_linear_forward(const uint16_t* X, int64_t T, int64_t ldx, const qg_qtensor* W, uint16_t* Y,
                                int64_t ldy, int32_t* status, void* stream) {
  int rc = check_qtensor(W, 8);
  if (rc != QG_OK) return rc;
  if (!linear_extent_ok(T) || !linear_extent_ok(W->rows) || !linear_extent_ok(W->cols)) return QG_UNSUPPORTED_SHAPE;
  if ((rc = check_bf16_matrix(X, T, W->cols, ldx)) != QG_OK) return rc;
  if ((rc = check_bf16_matrix(Y, T, W->rows, ldy)) != QG_OK) return rc;
  return launch_int8_linear(0, X, ldx, nullptr, 0, W, T, W->rows, W->cols, Y, ldy, status, (cudaStream_t)stream);
}

int qgalore_int8_linear_backward_input(const uint16_t* dY, int64_t T, int64_t lddy, const qg_qtensor* W,
                                       uint16_t* dX, int64_t lddx, int32_t* status, void* stream) {
  int rc = check_qtensor(W, 8);
  if (rc != QG_OK) return rc;
  if (!linear_extent_ok(T) || !linear_extent_ok(W->rows) || !linear_extent_ok(W->cols)) return QG_UNSUPPORTED_SHAPE;
  if ((rc = check_bf16_matrix(dY, T, W->rows, lddy)) != QG_OK) return rc;
  if ((rc = check_bf16_matrix(dX, T, W->cols, lddx)) != QG_OK) return rc;
  return launch_int8_linear(1, dY, lddy, nullptr, 0, W, T, W->rows, W->cols, dX, lddx, status, (cudaStream_t)stream);
}

int qgalore_int8_linear_backward_weight(const uint16_t* dY, int64_t T, int64_t lddy, const uint16_t* X, int64_t ldx,
                                        int64_t m, int64_t n, uint16_t* G, int64_t ldg, int32_t* status,
                                        void* stream) {
  if (!linear_extent_ok(T) || !linear_extent_ok(m) || !linear_extent_ok(n)) return QG_UNSUPPORTED_SHAPE;
  int rc;
  if ((rc = check_bf16_matrix(dY, T, m, lddy)) != QG_OK) return rc;
  if ((rc = check_bf16_matrix(X, T, n, ldx)) != QG_OK) return rc;
  if ((rc = check_bf16_matrix(G, m, n, ldg)) != QG_OK) return rc;
  // both operands are read in whole 64-column slabs: the row pitch has to cover the last one
  if (lddy < (m + 63) / 64 * 64 || ldx < (n + 63) / 64 * 64) return QG_UNSUPPORTED_SHAPE;
  return launch_int8_linear(2, dY, lddy, X, ldx, nullptr, T, m, n, G, ldg, status, (cudaStream_t)stream);
}

size_t qgalore_workspace_bytes(int op, int64_t m, int64_t n, int64_t r) {
  if (m <= 0 || r <= 0) return 0;
  switch (op) {
    case QG_OP_PROJECT_STEP: {
      if (n <= 0) return 0;
      // either projection side: the scratch holds P~ (rows of the projection x r) and N_b (r x columns of the state)
      const size_t a = simt_workspace_bytes(m, n, r), b = tc_workspace_bytes(m, n, r), c = tc_workspace_bytes(n, m, r);
      return a > b ? (a > c ? a : c) : (b > c ? b : c);
    }
    case QG_OP_REFRESH: {
      if (n <= 0) return 0;
      const size_t a = refresh_workspace_bytes(m, n, r), s = similarity_workspace_bytes(m, r);
      return a > s ? a : s;
    }
    case QG_OP_SIMILARITY: return similarity_workspace_bytes(m, r);
    default: return 0;
  }
}

static void fill_scalars(const qg_hyper* h, uint64_t seed, StepScalars* sc) {
  sc->beta1 = h->beta1; sc->beta2 = h->beta2;
  sc->one_minus_beta1 = 1.0f - h->beta1; sc->one_minus_beta2 = 1.0f - h->beta2;
  sc->bias1 = (float)(1.0 - std::pow((double)h->beta1, (double)h->step));
  sc->bias2 = (float)(1.0 - std::pow((double)h->beta2, (double)h->step));
  sc->eps = h->eps;
  sc->lr_alpha = (float)((double)h->lr * (double)h->alpha);
  sc->lr_wd = (float)((double)h->lr * (double)h->weight_decay);
  sc->seed_lo = (uint32_t)(seed & 0xFFFFFFFFull); sc->seed_hi = (uint32_t)(seed >> 32);
  sc->step_lo = (uint32_t)((uint64_t)h->step & 0xFFFFFFFFull); sc->step_hi = (uint32_t)((uint64_t)h->step >> 32);
  sc->rounding = h->rounding;
}

static int check_hyper(const qg_hyper* h) {
  if (!h || h->step < 1) return QG_INVALID_ARGUMENT;
  if (h->rounding != QG_ROUND_STOCHASTIC && h->rounding != QG_ROUND_NEAREST) return QG_INVALID_ARGUMENT;
  if (!std::isfinite(h->lr) || !(h->beta1 >= 0.f && h->beta1 < 1.f) || !(h->beta2 >= 0.f && h->beta2 < 1.f))
    return QG_INVALID_ARGUMENT;
  return QG_OK;
}

// Shape, pointer and alignment rules of one matrix of the step; fills everything of `a` but the scalars.
static int check_matrix(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r, const qg_qtensor* P,
                        const qg_qtensor* W, float* M, float* V, int64_t ldmv, int side, StepArgs* a, int state_bits = 0,
                        float* M_scale = nullptr, float* V_scale = nullptr) {
  if (!G || !M || !V) return QG_INVALID_ARGUMENT;
  if (side != QG_SIDE_LEFT && side != QG_SIDE_RIGHT) return QG_INVALID_ARGUMENT;
  const bool right = side == QG_SIDE_RIGHT;
  const int64_t prow = right ? n : m, scol = right ? m : n;     // rows of the projection, columns of the moments
  if (m <= 0 || n <= 0 || r <= 0 || ldg < n || ldmv < scol) return QG_INVALID_ARGUMENT;
  if (!P || (P->bits != 2 && P->bits != 4 && P->bits != 8)) return QG_INVALID_ARGUMENT;
  int rc = check_qtensor(P, P->bits);
  if (rc != QG_OK) return rc;
  rc = check_qtensor(W, 8);
  if (rc != QG_OK) return rc;
  if (P->rows != prow || P->cols != r || W->rows != m || W->cols != n) return QG_INVALID_ARGUMENT;
  if (r % 32 != 0 || r < 32 || r > 2048 || r > prow) return QG_UNSUPPORTED_SHAPE;
  if (m > (1ll << 31) - 1 || n > (1ll << 31) - 1) return QG_UNSUPPORTED_SHAPE;
  if (state_bits != 0 && state_bits != 32 && state_bits != 8) return QG_INVALID_ARGUMENT;
  const bool state8 = state_bits == 8;
  if (state8 && (!M_scale || !V_scale)) return QG_INVALID_ARGUMENT;
  if (!aligned16(G) || !aligned16(M) || !aligned16(V) || ldg % 8 != 0 || ldmv % (state8 ? 16 : 4) != 0) return QG_MISALIGNED;
  if (state8 && ((reinterpret_cast<uintptr_t>(M_scale) & 3u) || (reinterpret_cast<uintptr_t>(V_scale) & 3u))) return QG_MISALIGNED;
  memset(a, 0, sizeof(*a));
  a->G = G; a->ldg = ldg; a->m = m; a->n = n; a->r = r;
  a->P = *P; a->W = *W; a->M = M; a->V = V; a->ldmv = ldmv;
  a->right = right ? 1 : 0;
  a->state8 = state8 ? 1 : 0; a->M_scale = M_scale; a->V_scale = V_scale;
  return QG_OK;
}

static int project_step_impl(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r, const qg_qtensor* P,
                             const qg_qtensor* W, float* M, float* V, int64_t ldmv, const qg_hyper* h,
                             void* workspace, size_t workspace_bytes, int32_t* status_dev, const qg_debug* dbg,
                             void* stream, bool validate_only, int side = QG_SIDE_LEFT, int state_bits = 0,
                             float* M_scale = nullptr, float* V_scale = nullptr) {
  if (!workspace) return QG_INVALID_ARGUMENT;
  int rc = check_hyper(h);
  if (rc != QG_OK) return rc;
  StepArgs a;
  rc = check_matrix(G, ldg, m, n, r, P, W, M, V, ldmv, side, &a, state_bits, M_scale, V_scale);
  if (rc != QG_OK) return rc;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return QG_MISALIGNED;
  if (status_dev && (reinterpret_cast<uintptr_t>(status_dev) & 3u)) return QG_MISALIGNED;
  if (workspace_bytes < qgalore_workspace_bytes(QG_OP_PROJECT_STEP, m, n, r)) return QG_WORKSPACE_TOO_SMALL;
  if (validate_only) return QG_OK;
  a.ws = workspace; a.ws_bytes = workspace_bytes; a.status = status_dev;
  if (dbg) a.dbg = *dbg;
  fill_scalars(h, h->seed, &a.sc);
  if (g_step_impl == 1) {
    if (a.right || a.state8) return QG_UNSUPPORTED_SHAPE;   // the CUDA-core cross-check knows the left form, fp32 moments
    return launch_project_step_simt(a, (cudaStream_t)stream);
  }
  return launch_project_step_tc(a, (cudaStream_t)stream);
}

int qgalore_project_step(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r, const qg_qtensor* P,
                         const qg_qtensor* W, float* M, float* V, int64_t ldmv, const qg_hyper* h,
                         void* workspace, size_t workspace_bytes, int32_t* status_dev, const qg_debug* dbg,
                         void* stream) {
  return project_step_impl(G, ldg, m, n, r, P, W, M, V, ldmv, h, workspace, workspace_bytes, status_dev, dbg, stream,
                           false);
}

int qgalore_project_step_right(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r, const qg_qtensor* Q,
                               const qg_qtensor* W, float* Mt, float* Vt, int64_t ldmv, const qg_hyper* h,
                               void* workspace, size_t workspace_bytes, int32_t* status_dev, const qg_debug* dbg,
                               void* stream) {
  return project_step_impl(G, ldg, m, n, r, Q, W, Mt, Vt, ldmv, h, workspace, workspace_bytes, status_dev, dbg, stream,
                           false, QG_SIDE_RIGHT);
}

int qgalore_project_step_item(const qg_step_item* it, const qg_hyper* h, void* workspace, size_t workspace_bytes,
                              int32_t* status_dev, const qg_debug* dbg, void* stream) {
  if (!it || !h) return QG_INVALID_ARGUMENT;
  qg_hyper hi = *h;
  hi.seed = it->seed;
  return project_step_impl(it->G, it->ldg, it->m, it->n, it->r, &it->P, &it->W, it->M, it->V, it->ldmv, &hi, workspace,
                           workspace_bytes, status_dev, dbg, stream, false, it->side, it->state_bits, it->M_scale, it->V_scale);
}

size_t qgalore_workspace_bytes_batched(const qg_step_item* items, int32_t count) {
  size_t need = 0;
  if (!items) return 0;
  for (int32_t i = 0; i < count; ++i) {
    const size_t b = qgalore_workspace_bytes(QG_OP_PROJECT_STEP, items[i].m, items[i].n, items[i].r);
    need = b > need ? b : need;
  }
  return need;
}

int qgalore_project_step_batched(const qg_step_item* items, int32_t count, const qg_hyper* h, void* workspace,
                                 size_t workspace_bytes, int32_t* status_dev, void* stream) {
  if (!items || count <= 0 || !h) return QG_INVALID_ARGUMENT;
  // first pass validates everything (a dry run of the single-matrix checks), second pass enqueues
  for (int pass = 0; pass < 2; ++pass) {
    for (int32_t i = 0; i < count; ++i) {
      const qg_step_item& it = items[i];
      qg_hyper hi = *h;
      hi.seed = it.seed;
      const int rc = project_step_impl(it.G, it.ldg, it.m, it.n, it.r, &it.P, &it.W, it.M, it.V, it.ldmv, &hi,
                                       workspace, workspace_bytes, status_dev, nullptr, stream, pass == 0, it.side,
                                       it.state_bits, it.M_scale, it.V_scale);
      if (rc != QG_OK) return rc;
    }
  }
  return QG_OK;
}

struct qg_plan {
  Plan* impl;
};

static int plan_args(const qg_step_item* items, int32_t count, std::vector<StepArgs>* args) {
  args->resize((size_t)count);
  for (int32_t i = 0; i < count; ++i) {
    const qg_step_item& it = items[i];
    const int rc = check_matrix(it.G, it.ldg, it.m, it.n, it.r, &it.P, &it.W, it.M, it.V, it.ldmv, it.side, &(*args)[i],
                                it.state_bits, it.M_scale, it.V_scale);
    if (rc != QG_OK) return rc;
    (*args)[i].sc.seed_lo = (uint32_t)(it.seed & 0xFFFFFFFFull);
    (*args)[i].sc.seed_hi = (uint32_t)(it.seed >> 32);
  }
  return QG_OK;
}

size_t qgalore_plan_table_bytes(const qg_step_item* items, int32_t count) {
  if (!items || count <= 0) return 0;
  std::vector<StepArgs> args;
  if (plan_args(items, count, &args) != QG_OK) return 0;
  return plan_table_bytes(args.data(), count);
}

int qgalore_plan_create(const qg_step_item* items, int32_t count, void* table_dev, size_t table_bytes,
                        void* workspace, size_t workspace_bytes, qg_plan** plan) {
  if (!items || count <= 0 || !table_dev || !workspace || !plan) return QG_INVALID_ARGUMENT;
  if ((reinterpret_cast<uintptr_t>(workspace) & 1023u) || (reinterpret_cast<uintptr_t>(table_dev) & 255u))
    return QG_MISALIGNED;
  std::vector<StepArgs> args;
  const int rca = plan_args(items, count, &args);
  if (rca != QG_OK) return rca;
  Plan* impl = nullptr;
  const int rc = plan_create(args.data(), count, table_dev, table_bytes, workspace, workspace_bytes, &impl);
  if (rc != QG_OK) return rc;
  *plan = new qg_plan{impl};
  return QG_OK;
}

int qgalore_plan_step(const qg_plan* plan, const qg_hyper* h, int32_t* status_dev, void* stream) {
  if (!plan || !plan->impl) return QG_INVALID_ARGUMENT;
  const int rc = check_hyper(h);
  if (rc != QG_OK) return rc;
  if (status_dev && (reinterpret_cast<uintptr_t>(status_dev) & 3u)) return QG_MISALIGNED;
  StepScalars sc;
  fill_scalars(h, 0, &sc);
  return plan_step(plan->impl, sc, status_dev, (cudaStream_t)stream, nullptr);
}

int qgalore_plan_step_timed(const qg_plan* plan, const qg_hyper* h, int32_t* status_dev, void* stream,
                            float* kernel_ms, int32_t* kernel_launches) {
  if (!plan || !plan->impl || !kernel_ms || !kernel_launches) return QG_INVALID_ARGUMENT;
  const int rc = check_hyper(h);
  if (rc != QG_OK) return rc;
  StepScalars sc;
  fill_scalars(h, 0, &sc);
  return plan_step_timed(plan->impl, sc, status_dev, (cudaStream_t)stream, kernel_ms, kernel_launches);
}

void qgalore_plan_destroy(qg_plan* plan) {
  if (!plan) return;
  plan_destroy(plan->impl);
  delete plan;
}

// Argument rules of a refresh, for one matrix or a batch of one shape; on success enqueues everything.
static int refresh_impl(const qg_refresh_item* items, int32_t count, int64_t m, int64_t n, int64_t r, int32_t iters,
                        int32_t oversample_cols, int32_t sim_cols, void* workspace, size_t workspace_bytes,
                        int32_t* status_dev, void* stream, bool right) {
  if (!items || count <= 0 || !workspace || m <= 0 || n <= 0 || r <= 0 || iters < 0 || oversample_cols < 0)
    return QG_INVALID_ARGUMENT;
  // the matrix whose LEFT singular vectors are wanted: G, or G^T for the right-hand projection
  const int64_t pm = right ? n : m, pn = right ? m : n;
  const int64_t b = r + oversample_cols;
  // the block is handled in panels of 64 columns and cannot be wider than the matrix is tall or wide
  if (r % 32 != 0 || b % 64 != 0 || b > m || b > n || b > 4096 || m > (1ll << 31) - 1 || n > (1ll << 31) - 1)
    return QG_UNSUPPORTED_SHAPE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return QG_MISALIGNED;
  if (status_dev && (reinterpret_cast<uintptr_t>(status_dev) & 3u)) return QG_MISALIGNED;
  std::vector<RefreshJob> jobs((size_t)count);
  for (int32_t i = 0; i < count; ++i) {
    const qg_refresh_item& it = items[i];
    if (!it.G || it.ldg < n || it.ldg != items[0].ldg) return QG_INVALID_ARGUMENT;
    int rc = check_projection_qtensor(&it.P_new);
    if (rc != QG_OK) return rc;
    if (it.P_new.rows != pm || it.P_new.cols != r || it.P_new.ld != r) return QG_INVALID_ARGUMENT;
    if (it.P_prev) {
      rc = check_projection_qtensor(it.P_prev);
      if (rc != QG_OK) return rc;
      if (it.P_prev->rows != pm || it.P_prev->cols != r) return QG_INVALID_ARGUMENT;
    }
    if (!aligned16(it.G) || it.ldg % 8 != 0) return QG_MISALIGNED;
    if (it.P_fp32 && !aligned16(it.P_fp32)) return QG_MISALIGNED;
    if (it.sim_dev && !aligned4(it.sim_dev)) return QG_MISALIGNED;
    jobs[(size_t)i] = RefreshJob{it.G, it.ldg, it.seed, &it.P_new, it.P_fp32};
  }
  if (workspace_bytes < qgalore_workspace_bytes(QG_OP_REFRESH, pm, pn, b)) return QG_WORKSPACE_TOO_SMALL;
  constexpr int kJacobiSweeps = 12;
  int rc = launch_refresh_batched(jobs.data(), count, pm, pn, r, b, iters, kJacobiSweeps, workspace, workspace_bytes, status_dev,
                                  (cudaStream_t)stream, right);
  if (rc != QG_OK) return rc;
  for (int32_t i = 0; i < count; ++i) {
    const qg_refresh_item& it = items[i];
    if (it.P_prev && it.sim_dev) {
      const int32_t c = (sim_cols <= 0 || sim_cols > r) ? (int32_t)r : sim_cols;
      // the refresh has finished with its scratch by the time this runs on the same stream
      rc = launch_similarity(it.P_prev, &it.P_new, c, it.sim_dev, workspace, (cudaStream_t)stream);
      if (rc != QG_OK) return rc;
    }
  }
  return QG_OK;
}

static int refresh_single(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r, int32_t iters,
                          int32_t oversample_cols, uint64_t seed, const qg_qtensor* P_new, float* P_fp32,
                          const qg_qtensor* P_prev, int32_t sim_cols, float* sim_dev, void* workspace,
                          size_t workspace_bytes, int32_t* status_dev, void* stream, bool right) {
  if (!P_new) return QG_INVALID_ARGUMENT;
  const qg_refresh_item item{G, ldg, seed, *P_new, P_fp32, P_prev, sim_dev};
  return refresh_impl(&item, 1, m, n, r, iters, oversample_cols, sim_cols, workspace, workspace_bytes, status_dev, stream, right);
}

int qgalore_refresh_subspace_batched(const qg_refresh_item* items, int32_t count, int64_t m, int64_t n, int64_t r,
                                     int32_t iters, int32_t oversample_cols, int32_t side, int32_t sim_cols, void* workspace,
                                     size_t workspace_bytes, int32_t* status_dev, void* stream) {
  if (side != QG_SIDE_LEFT && side != QG_SIDE_RIGHT) return QG_INVALID_ARGUMENT;
  return refresh_impl(items, count, m, n, r, iters, oversample_cols, sim_cols, workspace, workspace_bytes, status_dev, stream,
                      side == QG_SIDE_RIGHT);
}

int qgalore_refresh_subspace(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r, int32_t iters,
                             int32_t oversample_cols, uint64_t seed, const qg_qtensor* P_new, float* P_fp32,
                             const qg_qtensor* P_prev, int32_t sim_cols, float* sim_dev, void* workspace,
                             size_t workspace_bytes, int32_t* status_dev, void* stream) {
  return refresh_single(G, ldg, m, n, r, iters, oversample_cols, seed, P_new, P_fp32, P_prev, sim_cols, sim_dev, workspace,
                        workspace_bytes, status_dev, stream, false);
}

int qgalore_refresh_subspace_right(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r, int32_t iters,
                                   int32_t oversample_cols, uint64_t seed, const qg_qtensor* Q_new, float* Q_fp32,
                                   const qg_qtensor* Q_prev, int32_t sim_cols, float* sim_dev, void* workspace,
                                   size_t workspace_bytes, int32_t* status_dev, void* stream) {
  return refresh_single(G, ldg, m, n, r, iters, oversample_cols, seed, Q_new, Q_fp32, Q_prev, sim_cols, sim_dev, workspace,
                        workspace_bytes, status_dev, stream, true);
}

int qgalore_subspace_similarity(const qg_qtensor* A, const qg_qtensor* B, int32_t sim_cols, float* sim_dev,
                                void* workspace, size_t workspace_bytes, void* stream) {
  if (!sim_dev || !workspace) return QG_INVALID_ARGUMENT;
  int rc = check_projection_qtensor(A);
  if (rc != QG_OK) return rc;
  rc = check_projection_qtensor(B);
  if (rc != QG_OK) return rc;
  if (A->rows != B->rows || A->cols != B->cols) return QG_INVALID_ARGUMENT;
  if (!aligned4(sim_dev)) return QG_MISALIGNED;
  const int32_t c = (sim_cols <= 0 || sim_cols > A->cols) ? (int32_t)A->cols : sim_cols;
  if (A->cols > 16384) return QG_UNSUPPORTED_SHAPE;
  if (workspace_bytes < similarity_workspace_bytes(A->rows, A->cols)) return QG_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(workspace) & 15u) return QG_MISALIGNED;
  return launch_similarity(A, B, c, sim_dev, workspace, (cudaStream_t)stream);
}

int qgalore_gate_update(float sim, float threshold, int32_t k, int32_t* interval, float* history, int32_t* count) {
  if (k < 1 || !interval || !history || !count || *count < 0 || *count > k || *interval < 1) return QG_INVALID_ARGUMENT;
  if (*count == k) {                       // keep the last k values
    for (int i = 1; i < k; ++i) history[i - 1] = history[i];
    *count = k - 1;
  }
  history[(*count)++] = sim;
  if (*count < k) return 0;
  for (int i = 0; i < k; ++i)
    if (!(history[i] >= threshold)) return 0;
  if (*interval > (1 << 29)) return 0;     // never overflow the interval
  *interval *= 2;
  *count = 0;
  return 1;
}

int qgalore_debug_kernel_info(char* buf, size_t capacity) {
  if (!buf || capacity < 2) return QG_INVALID_ARGUMENT;
  buf[0] = 0;
  return tc_kernel_info(buf, capacity);
}

int qgalore_debug_set_pair_mode(int mask) { return set_pair_mode(mask); }
int qgalore_debug_set_fused_dequant(int on) { return set_fused_dequant(on); }
int qgalore_debug_set_refresh_tensor_cores(int on) { return set_refresh_tc(on); }
int qgalore_debug_set_jacobi_blocks(int on) { return set_jacobi_blocks(on); }
int qgalore_debug_set_chunk_budget(size_t bytes) { return bytes >= (1u << 20) ? set_chunk_budget(bytes) : QG_INVALID_ARGUMENT; }

/* Test aid: selects the CUDA-core (1) or the tensor-core (0) kernels of qgalore_project_step. */
int qgalore_debug_set_step_impl(int impl) {
  if (impl != 0 && impl != 1) return QG_INVALID_ARGUMENT;
  g_step_impl = impl;
  return QG_OK;
}

}  // extern "C"
