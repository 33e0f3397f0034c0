/*
 * qgalore.h - C boundary of the B200 (sm_100a) Q-GaLore per-step optimizer library.
 *
 * Q-GaLore (arXiv 2407.08296) keeps each weight matrix W (m x n) in INT8, the GaLore
 * projection matrix P (m x r) in INT4, and the Adam moments M, V (r x n) of the projected
 * gradient in the low-rank space.  One optimizer step of one matrix is (Sec. 3.5):
 *
 *     P~ = dequant(P)            R = P~^T G          (project the bf16 gradient)
 *     M, V <- Adam(M, V, R)      N = M^ / (sqrt(V^) + eps)
 *     W' = dequant(W) - lr * alpha * P~ N            (project back, scale)
 *     W  <- Quant_8 with stochastic rounding (W')    (Sec. 3.4)
 *
 * Common rules for every entry point
 *   - Return value: 0 (QG_OK) or a negative qg_status.  No exceptions, no allocation, no
 *     implicit synchronisation: work is enqueued on the caller's stream (a cudaStream_t passed
 *     as void*, NULL = the default stream) and the call returns.
 *   - Unless stated otherwise every buffer is DEVICE memory owned by the caller; the library
 *     neither frees nor retains it.  Structs (qg_qtensor, qg_hyper) are HOST memory read
 *     during the call.
 *   - Matrices are row-major with a row pitch ("ld") in ELEMENTS.  Base pointers must be
 *     16-byte aligned and every row pitch a multiple of 16 bytes, i.e. ld % 8 == 0 for bf16,
 *     ld % 4 == 0 for fp32, ld % 16 == 0 for INT8 codes, ld % 32 == 0 for INT4, ld % 64 == 0 for INT2 codes.
 *     Elements between cols and ld are padding: never read as data, never written.
 *   - Quantization groups (Sec. 3.1, "block-wise", block 256) are runs of `group` consecutive
 *     elements along a row and restart at every row; a row whose length is not a multiple of
 *     `group` ends in one shorter group.  scales/zeros are dense [rows][ceil(cols/group)] fp32.
 *   - INT4 codes are packed two per byte: byte k of a row holds column 2k in its low nibble
 *     and column 2k+1 in its high nibble, each stored as code + 8 (codes lie in [-8, 7]).
 *     INT2 codes (the 2-bit projection of the ablation in Sec. 4.4) are packed four per byte:
 *     column 4k + i of a row sits in bits 2i, 2i + 1 of byte k, stored as code + 2 (codes in [-2, 1]).
 *   - A device status word (int32, optional, may be NULL) is OR-ed with QG_DEV_* flags when a
 *     kernel gives up a bounded wait or an iteration does not converge; it is never cleared
 *     by the library.
 */
#ifndef QGALORE_H_
#define QGALORE_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define QG_API __attribute__((visibility("default")))
#else
#define QG_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  QG_OK = 0,
  QG_INVALID_ARGUMENT = -1,    /* null pointer, non-positive size, bits/group not supported   */
  QG_UNSUPPORTED_SHAPE = -2,   /* r > m, r not a multiple of 32, r > 2048, size beyond a limit */
  QG_MISALIGNED = -3,          /* base pointer or row pitch breaks the 16-byte rule            */
  QG_WORKSPACE_TOO_SMALL = -4,
  QG_CUDA_ERROR = -5,          /* a CUDA runtime/driver call failed; see qgalore_last_cuda_error */
  QG_NOT_CONVERGED = -6
} qg_status;

/* flags OR-ed into the optional device status word */
#define QG_DEV_WAIT_EXPIRED 1   /* a bounded barrier wait ran out; the tile was abandoned */
#define QG_DEV_NOT_CONVERGED 2  /* eigen-iteration of the refresh hit its sweep limit     */
#define QG_DEV_BAD_FACTOR 4     /* Cholesky factor of the refresh met a non-positive pivot */

/* A block-wise quantized matrix (Sec. 3.1; App. A: W = (codes - zeros) * scales). */
typedef struct {
  void*   codes;   /* device; bits == 8: int8 [rows][ld]; 4: uint8 [rows][ld / 2]; 2: uint8 [rows][ld / 4] */
  float*  scales;  /* device; [rows][ceil(cols / group)]                                    */
  float*  zeros;   /* device; same shape, integer valued                                    */
  int64_t rows, cols, ld;
  int32_t bits;    /* 8 (weights, projection), 4 (projection, the method), 2 (projection)   */
  int32_t group;   /* 256                                                                   */
} qg_qtensor;

/* Hyper-parameters of one step.  alpha is GaLore's scale factor (0.25 in Sec. 4.1), the
 * Adam constants are Kingma & Ba's; step is t >= 1 and enters the bias corrections and the
 * random-number counter; seed keys the stochastic rounding of this matrix.  rounding selects how
 * the updated weight is requantized: QG_ROUND_STOCHASTIC (Sec. 3.4, the method) or QG_ROUND_NEAREST
 * (the ablation of Sec. 4.4, Fig. 6: round to nearest, ties to even; seed and step do not enter the codes). */
#define QG_ROUND_STOCHASTIC 0
#define QG_ROUND_NEAREST 1
typedef struct {
  float    lr, alpha, beta1, beta2, eps, weight_decay;
  int64_t  step;
  uint64_t seed;
  int32_t  rounding;   /* QG_ROUND_*; anything else: QG_INVALID_ARGUMENT */
  int32_t  reserved;   /* 0 */
} qg_hyper;

/* Optional taps for tests: any non-null pointer receives that intermediate (device, fp32). */
typedef struct {
  float* R;      /* r x n, pitch ldmv: projected gradient                     */
  float* N;      /* r x n, pitch ldmv: Adam direction before bfloat16 rounding */
  float* W_pre;  /* m x n, pitch W->ld: weight before requantization           */
  uint16_t* N_b; /* r x n, pitch ldmv (elements): the bfloat16 direction as the back-projection reads it */
} qg_debug;

/* --- Sec. 3.1 / Sec. 3.3: round-to-nearest block-wise quantization ----------------------
 * dst->codes/scales/zeros receive Quant_4 (resp. Quant_8) of src (fp32, rows x cols, pitch
 * ld_src).  Per group: s = (max - min) / (2^bits - 1), z = -2^(bits-1) - rint(min / s),
 * code = clamp(rint(x / s) + z); x / s is evaluated as x * (1 / s) in binary32, ties to even.
 * A constant group takes z = 0, s = |max| (1 if that is 0).  dst->rows/cols must equal
 * rows/cols, dst->bits must be 4 (resp. 8, 2).  Bit-exact against the CPU oracle.
 * qgalore_quantize_int2 is Quant_2, for the 2-bit projection of the ablation in Sec. 4.4 (Fig. 3). */
QG_API int qgalore_quantize_int4(const float* src, int64_t rows, int64_t cols, int64_t ld_src,
                          const qg_qtensor* dst, void* stream);
QG_API int qgalore_quantize_int2(const float* src, int64_t rows, int64_t cols, int64_t ld_src,
                          const qg_qtensor* dst, void* stream);
QG_API int qgalore_quantize_int8(const float* src, int64_t rows, int64_t cols, int64_t ld_src,
                          const qg_qtensor* dst, void* stream);

/* App. A, dequantization line: dst (fp32, pitch ld_dst) = (codes - zeros) * scales. */
QG_API int qgalore_dequantize(const qg_qtensor* src, float* dst, int64_t ld_dst, void* stream);

/* --- Sec. 3.5 (with Sec. 3.4 for the write-back): one optimizer step of one matrix ------
 * G       bf16 bit patterns, m x n, pitch ldg                        (read)
 * P       INT4 (the method; INT2 or INT8 for the ablation of Sec. 4.4), m x r   (read)
 * W       INT8, m x n: codes, scales and zeros are replaced          (read + write)
 * M, V    fp32, r x n, pitch ldmv                                    (read + write)
 * h       host; step >= 1
 * workspace  device scratch of at least qgalore_workspace_bytes(QG_OP_PROJECT_STEP, m, n, r)
 *            bytes, 256-byte aligned; contents are undefined afterwards
 * status_dev optional device status word
 * dbg     optional (may be NULL) test taps
 * Shape limits: 32 <= r <= 2048, r % 32 == 0, r <= m.  Errors are reported before anything
 * is enqueued; after QG_OK the work is queued on `stream`. */
QG_API int qgalore_project_step(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r,
                         const qg_qtensor* P, const qg_qtensor* W,
                         float* M, float* V, int64_t ldmv, const qg_hyper* h,
                         void* workspace, size_t workspace_bytes,
                         int32_t* status_dev, const qg_debug* dbg, void* stream);

/* --- Sec. 3.5 with the projection on the right (the paper takes GaLore's projection, which projects
 * on the side of the shorter dimension): R = G Q with Q n x r, Adam on the m x r state, D = N Q^T.
 * Q       INT4 (or INT2 / INT8), n x r                                (read)
 * Mt, Vt  fp32, the m x r moments stored TRANSPOSED: r x m, pitch ldmv >= m   (read + write)
 * dbg->R, dbg->N (if given) are r x m too.  Everything else as in qgalore_project_step; r <= n.
 * In a plan or a batched call an item selects this form with side = QG_SIDE_RIGHT. */
#define QG_SIDE_LEFT 0
#define QG_SIDE_RIGHT 1
QG_API int qgalore_project_step_right(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r,
                               const qg_qtensor* Q, const qg_qtensor* W,
                               float* Mt, float* Vt, int64_t ldmv, const qg_hyper* h,
                               void* workspace, size_t workspace_bytes,
                               int32_t* status_dev, const qg_debug* dbg, void* stream);

/* --- Sec. 3.5, the same step for several matrices (a layer, or a whole stack) in one call ----
 * Every item is one independent matrix with its own buffers and its own stochastic-rounding
 * seed; lr, alpha, the Adam constants and the step index come from h (h->seed is ignored).
 * items is HOST memory.  The workspace (qgalore_workspace_bytes_batched) is shared by the
 * items, which are processed in order on `stream`, three launches per matrix.  Validation covers
 * every item before anything is enqueued.  This call is for lists that change from call to call;
 * a list that is stepped repeatedly belongs in a plan (below), which prepares the descriptors once
 * and runs a whole chunk of matrices per launch (LLaMA-1B stack: 3.2 ms per step as a plan). */
typedef struct {
  const uint16_t* G; int64_t ldg, m, n, r;
  qg_qtensor P, W;
  float* M; float* V; int64_t ldmv;
  uint64_t seed;
  int32_t side;       /* QG_SIDE_LEFT (0) or QG_SIDE_RIGHT: see qgalore_project_step_right */
  int32_t state_bits; /* 0 or 32: M, V are fp32.  8: the 8-bit block-wise storage below */
  float* M_scale;     /* state_bits == 8 only: fp32 scales, dense [r][ceil(cols / 32)], cols = n (left) or m (right) */
  float* V_scale;
} qg_step_item;

/* 8-bit moments (Sec. 3.5 keeps the Adam states in 8 bits and names no format; this one is the library's own).
 * With state_bits == 8, M points to int8 and V to uint8 codes, r x cols with a pitch of ldmv BYTES (a multiple
 * of 16).  Blocks are runs of 32 consecutive columns of a row (a shorter one at a ragged end), one scale each:
 *   M: scale s = max |x| of the block, code = rint(x / (s / 127)),              x^ = code * (s / 127)
 *   V: scale s = max x,               code = rint(255 * sqrt(x / s)),           x^ = (code / 255)^2 * s
 * (divisions by a scale are multiplications by its binary32 reciprocal; a zero block has scale 0, codes 0).
 * A step dequantizes the old moments, updates them and takes the direction in fp32, and stores the new ones. */

/* One item of the table above as a call of its own: any side, any moment storage.  dbg as in
 * qgalore_project_step (R, N have the shape of the moments). */
QG_API int qgalore_project_step_item(const qg_step_item* item, const qg_hyper* h, void* workspace, size_t workspace_bytes,
                              int32_t* status_dev, const qg_debug* dbg, void* stream);

QG_API int qgalore_project_step_batched(const qg_step_item* items, int32_t count, const qg_hyper* h,
                                 void* workspace, size_t workspace_bytes,
                                 int32_t* status_dev, void* stream);
QG_API size_t qgalore_workspace_bytes_batched(const qg_step_item* items, int32_t count);

/* --- Sec. 3.5, the step of a fixed list of matrices prepared once ("plan") -------------------------
 * A training loop steps the same matrices, in the same buffers, thousands of times.  A plan does the
 * per-matrix set-up once (validation, TMA descriptors, tile tables) and then steps the whole list with
 * a few grouped kernel launches: consecutive items are packed into chunks that share the workspace, and
 * each chunk runs as one dequantize-P launch, one projection+Adam launch and one back-projection+
 * requantization launch over all of its matrices.
 *   items       HOST; every buffer an item names must stay where it is while the plan lives
 *   table_dev   DEVICE, 256-byte aligned, qgalore_plan_table_bytes(items, count) bytes, owned by the caller and
 *               left untouched by it until qgalore_plan_destroy
 *   workspace   DEVICE scratch, 1024-byte aligned, at least qgalore_workspace_bytes_batched(items, count)
 *               bytes; more lets a chunk hold more matrices.  Contents are undefined between steps, but
 *               the buffer must not move.
 * qgalore_plan_create copies the table to the device synchronously; it allocates host memory only.
 * qgalore_plan_step enqueues one optimizer step of every matrix (lr, alpha, the Adam constants and the
 * step index from h; the stochastic-rounding seed of each matrix from its item) and returns. */
typedef struct qg_plan qg_plan;
QG_API size_t qgalore_plan_table_bytes(const qg_step_item* items, int32_t count);  /* 0 if an item is invalid */
QG_API int qgalore_plan_create(const qg_step_item* items, int32_t count, void* table_dev, size_t table_bytes,
                        void* workspace, size_t workspace_bytes, qg_plan** plan);
QG_API int qgalore_plan_step(const qg_plan* plan, const qg_hyper* h, int32_t* status_dev, void* stream);
QG_API void qgalore_plan_destroy(qg_plan* plan);
/* Measurement aid: the same step as qgalore_plan_step with a CUDA event recorded before and after every
 * kernel launch on `stream`; waits for the step to finish (the one entry point that synchronises, and
 * that creates and destroys events).  kernel_ms[0..2] (HOST) receive the summed device time of the
 * dequantize-P, projection+Adam and back-projection+requantize launches, kernel_launches[0..2] their counts. */
QG_API int qgalore_plan_step_timed(const qg_plan* plan, const qg_hyper* h, int32_t* status_dev, void* stream,
                            float* kernel_ms, int32_t* kernel_launches);

/* --- Sec. 3.5 "obtain the projection matrix using SVD" + Sec. 3.3 INT4 storage ------------
 * Top-r left singular vectors of G (bf16, m x n, pitch ldg) by block subspace iteration on G G^T with a
 * block of b = r + oversample_cols columns (`iters` multiplications by G G^T, each followed by a block
 * Gram-Schmidt orthonormalisation) and a Rayleigh-Ritz step (eigenvectors of the projected b x b matrix by
 * a Jacobi iteration on binary32 rows with binary64 sums), then Quant_4 into P_new.  Each column carries the sign that makes its
 * largest-magnitude entry positive.
 *   P_new      INT4, m x r, ld == r; written
 *   P_fp32     optional (may be NULL): m x r fp32, pitch r, receives the vectors before quantization
 *   P_prev, sim_dev  if both given, the similarity of Sec. 3.2 between P_prev and P_new over the leading
 *              sim_cols columns (<= 0: all) is written to *sim_dev
 *   workspace  qgalore_workspace_bytes(QG_OP_REFRESH, m, n, b) bytes, 256-byte aligned
 *   status_dev optional; receives QG_DEV_NOT_CONVERGED / QG_DEV_BAD_FACTOR
 * Shape rules: r % 32 == 0, b % 64 == 0, b <= min(m, n), b <= 4096.  Typical use: b = 2 r, iters = 12.
 * The Adam moments and the step count are not touched.  The random start block is drawn from Philox
 * keyed by `seed`. */
QG_API int qgalore_refresh_subspace(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r,
                             int32_t iters, int32_t oversample_cols, uint64_t seed,
                             const qg_qtensor* P_new, float* P_fp32,
                             const qg_qtensor* P_prev, int32_t sim_cols, float* sim_dev,
                             void* workspace, size_t workspace_bytes,
                             int32_t* status_dev, void* stream);
/* The same for the right-hand projection: the top-r RIGHT singular vectors of G, i.e. the left ones of G^T
 * (G is read with its strides swapped, nothing is transposed in memory).  Q_new, Q_prev, Q_fp32 are n x r;
 * workspace qgalore_workspace_bytes(QG_OP_REFRESH, n, m, b). */
QG_API int qgalore_refresh_subspace_right(const uint16_t* G, int64_t ldg, int64_t m, int64_t n, int64_t r,
                                   int32_t iters, int32_t oversample_cols, uint64_t seed,
                                   const qg_qtensor* Q_new, float* Q_fp32,
                                   const qg_qtensor* Q_prev, int32_t sim_cols, float* sim_dev,
                                   void* workspace, size_t workspace_bytes,
                                   int32_t* status_dev, void* stream);

/* --- Sec. 3.5, the refresh of several matrices of ONE shape in one call (with a fixed interval every matrix of a
 * stack is due in the same step; under the adaptive schedule of Sec. 3.2, those whose interval has run out).
 * The matrices are refreshed in batches: every kernel launch, and every grid barrier of the eigen-iteration,
 * serves all matrices of a batch, so that a stack costs far less than its matrices one after the other.
 *   items      HOST; per matrix: the gradient and its pitch, the seed of its start block, where the new
 *              projection goes (P_new, ld == r) and optionally the fp32 vectors (P_fp32), the previous projection
 *              (P_prev, may be NULL) and the device word that receives the similarity to it (sim_dev, may be NULL)
 *   m, n, r    the shape and rank all items share; ldg must be the same for all items as well
 *   side       QG_SIDE_LEFT: top-r left singular vectors (P_new is m x r); QG_SIDE_RIGHT: right ones (n x r)
 *   workspace  at least qgalore_workspace_bytes(QG_OP_REFRESH, ...) bytes (the extents as for the single-matrix
 *              call); a batch holds as many matrices as fit (up to 8), so count times that amount is the useful
 *              maximum.  256-byte aligned.
 * Results are those of the single-matrix call on each item (same seed, same arithmetic, bit for bit). */
typedef struct {
  const uint16_t* G; int64_t ldg;
  uint64_t seed;
  qg_qtensor P_new;
  float* P_fp32;
  const qg_qtensor* P_prev;
  float* sim_dev;
} qg_refresh_item;
QG_API int qgalore_refresh_subspace_batched(const qg_refresh_item* items, int32_t count, int64_t m, int64_t n, int64_t r,
                                     int32_t iters, int32_t oversample_cols, int32_t side, int32_t sim_cols,
                                     void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);

/* --- Sec. 3.2: cosine similarity between adjacent projection matrices -------------------
 * *sim_dev = sum_{j < c} |<a_j, b_j>| / (||A[:, :c]||_F ||B[:, :c]||_F), c = sim_cols
 * (<= 0 means all columns), on the dequantized INT4 matrices A and B (same shape).
 * workspace: qgalore_workspace_bytes(QG_OP_SIMILARITY, rows, 0, cols) bytes. */
QG_API int qgalore_subspace_similarity(const qg_qtensor* A, const qg_qtensor* B, int32_t sim_cols,
                                float* sim_dev, void* workspace, size_t workspace_bytes,
                                void* stream);

/* --- The same statistic for callers that cannot allocate device memory (the paper has no counterpart: this
 * is a convenience of the library).  Some code that wants the similarity runs where cudaMalloc is
 * not an option: inside a framework's optimizer hook that must not touch the caching allocator, in a process
 * whose memory budget was handed out up front, or on a stream that is being recorded.  For them the scratch
 * of the two reduction kernels sits in a fixed array inside the library instead of a caller workspace, so
 * the call takes only its inputs and the output scalar and never calls cudaMalloc, cudaFree or any
 * allocating routine.
 *   - Limit: qgalore_workspace_bytes(QG_OP_SIMILARITY, rows, 0, cols) must not exceed
 *     qgalore_subspace_similarity_static_max_bytes() (2 MiB: e.g. 11008 x 1024 fits, 16384 x 2048 does not);
 *     larger shapes return QG_WORKSPACE_TOO_SMALL and enqueue nothing.  Every GPU on which the library is
 *     loaded keeps those 2 MiB reserved until the process ends.
 *   - The first call on each device looks up the array's device address (a runtime query, made with that
 *     device current); make that first call before you start capturing a stream.
 *   - All calls on a device share the one array.  Nothing in it has to be zero on entry (the first kernel
 *     rewrites every word the second reads), but two calls that overlap on the GPU - different streams, or
 *     different host threads - race on it and return garbage: serialise them.
 * Results are identical to qgalore_subspace_similarity on the same inputs. */
QG_API int qgalore_subspace_similarity_static(const qg_qtensor* A, const qg_qtensor* B, int32_t sim_cols,
                                       float* sim_dev, void* stream);
QG_API size_t qgalore_subspace_similarity_static_max_bytes(void);

/* --- Sec. 3.2, adaptive lazy update: host-only state machine ----------------------------
 * Pushes `sim` into `history` (k floats, host) holding *count values; when k values are held
 * and all are >= threshold, *interval is doubled and the history cleared.  Returns 1 if the
 * interval was doubled, 0 if not, negative on bad arguments. */
QG_API int qgalore_gate_update(float sim, float threshold, int32_t k, int32_t* interval,
                        float* history, int32_t* count);

/* --- App. A: the INT8 linear layer (the products either side of the optimizer step) ------
 * W~ = bfloat16((codes - zeros) * scales): the INT8 weight (m x n, groups of 256 along a row) dequantized in
 * binary32 and rounded once to bfloat16 while its tiles enter the GEMM; it is never written to global memory.
 * All matrices are bfloat16 bit patterns, row-major, DEVICE memory; base pointers 16-byte aligned, row
 * pitches multiples of 8 elements; accumulation is binary32, the result is rounded once to bfloat16.
 * The listing's bias term is left out (the LLaMA layers have none).  W is only read.
 *   forward          Y  (T x m, pitch ldy)  = X  (T x n, pitch ldx)  * W~^T
 *   backward_input   dX (T x n, pitch lddx) = dY (T x m, pitch lddy) * W~
 *   backward_weight  G  (m x n, pitch ldg)  = dY^T * X     - the gradient qgalore_project_step consumes; no
 *                    quantized operand.  dY and X are read in whole 64-column slabs: lddy >= m and ldx >= n
 *                    rounded up to multiples of 64 (what lies in the padding does not matter), else
 *                    QG_UNSUPPORTED_SHAPE.
 * status (device int32, may be null) receives QG_DEV_WAIT_EXPIRED if a bounded wait ran out.  Extents up to
 * 2^30 and at most 2^30 output tiles of 128 x 256, else QG_UNSUPPORTED_SHAPE.  No workspace. */
QG_API int qgalore_int8_linear_forward(const uint16_t* X, int64_t T, int64_t ldx, const qg_qtensor* W,
                                uint16_t* Y, int64_t ldy, int32_t* status, void* stream);
QG_API int qgalore_int8_linear_backward_input(const uint16_t* dY, int64_t T, int64_t lddy, const qg_qtensor* W,
                                       uint16_t* dX, int64_t lddx, int32_t* status, void* stream);
QG_API int qgalore_int8_linear_backward_weight(const uint16_t* dY, int64_t T, int64_t lddy, const uint16_t* X,
                                        int64_t ldx, int64_t m, int64_t n, uint16_t* G, int64_t ldg,
                                        int32_t* status, void* stream);

enum { QG_OP_PROJECT_STEP = 1, QG_OP_REFRESH = 2, QG_OP_SIMILARITY = 3 };

/* Scratch bytes the given operation needs for an m x n matrix at rank r (host, pure).
 * For QG_OP_REFRESH r is the block width (rank + oversample_cols). */
QG_API size_t qgalore_workspace_bytes(int op, int64_t m, int64_t n, int64_t r);

QG_API const char* qgalore_status_string(int status);
/* Text of the last CUDA error this thread met inside the library ("" if none). */
QG_API const char* qgalore_last_cuda_error(void);
/* A tag that changes whenever the kernels of the optimizer step change in a way that can move their memory traffic
 * or timing; profiler figures taken on one revision are not quoted for another. */
QG_API const char* qgalore_kernel_revision(void);
/* Number of kernels the library has launched from this process (for launch accounting). */
QG_API uint64_t qgalore_launch_count(void);
/* --- Test aids.  Declared only when QGALORE_TEST_API is defined before this header is included: they are
 * process-global switches (not thread safe) that change what later calls do, meant for the test suite. ---- */
#ifdef QGALORE_TEST_API
/* 0 selects the tensor-core kernels of qgalore_project_step (the default and the product path), 1 the plain
 * CUDA-core kernels kept to cross-check them. */
QG_API int qgalore_debug_set_step_impl(int impl);
/* Which kernels of plans created after this call run as CTA pairs (tcgen05 cta_group::2, 256 x 256 tiles per
 * pair): bit 0 the back-projection (chunks of left-hand items only), bit 1 the projection (where every rank of a
 * chunk is a multiple of 256), bit 2 the back-projection in chunks whose ranks average 1024 or more.  0 = one CTA
 * per 128 x 256 tile; the default is 6.  Every setting gives the same results bit for bit. */
QG_API int qgalore_debug_set_pair_mode(int mask);
/* 1: the projection kernel converts the INT4 codes of P inside its main loop (converter warps write the bf16
 * operand tile straight into shared memory); 0 (the default, the faster arrangement as measured): P is dequantized
 * to bf16 by a separate grouped launch first, as for 2- and 8-bit codes.  Applies to calls and plans made
 * afterwards; the results are the same bit for bit. */
QG_API int qgalore_debug_set_fused_dequant(int on);
/* 1 (the default): the early iterations of a refresh take their two products with the gradient on the tensor cores
 * (the iterate split into three bfloat16 planes); 0: every product on the CUDA cores. */
QG_API int qgalore_debug_set_refresh_tensor_cores(int on);
/* 1 (the default): the eigen-iteration of a refresh handles the rows of the projected matrix in blocks of eight
 * kept in shared memory and registers (block widths up to 2048); 0: row by row through L2, the form wider blocks
 * take.  Applies to calls made afterwards; both meet the same accuracy bound, their results differ in the last bits. */
QG_API int qgalore_debug_set_jacobi_blocks(int on);
/* Scratch bytes a chunk of a plan may use (plans created afterwards; at least 1 MiB).  Larger chunks mean
 * fewer, longer launches; smaller ones keep the bf16 direction between the two kernels inside L2. */
QG_API int qgalore_debug_set_chunk_budget(size_t bytes);
/* Runs the bounded barrier wait every tensor-core kernel uses on a barrier that nothing ever signals, with a
 * limit of `polls` polls (1 .. 2^20), in one small kernel that has no copy in flight and holds no tensor
 * memory: the wait gives up, the kernel ORs QG_DEV_WAIT_EXPIRED into *status_dev and returns normally.
 * polls_used_dev (device, optional) receives the number of polls made. */
QG_API int qgalore_debug_expire_wait(int32_t polls, int32_t* status_dev, int32_t* polls_used_dev, void* stream);
#endif

/* Diagnostic: writes one text line per tensor-core kernel (registers per thread, thread limit, shared
 * memory) as the CUDA runtime reports them for the current device into buf (HOST, NUL-terminated). */
QG_API int qgalore_debug_kernel_info(char* buf, size_t capacity);

#ifdef __cplusplus
}
#endif
#endif /* QGALORE_H_ */
