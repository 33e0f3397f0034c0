// Placeholders for entry points whose kernels are not written yet.
#include "qg_common.cuh"
namespace qg {
int launch_project_step_simt(const StepArgs& a, cudaStream_t st);
size_t simt_workspace_bytes(int64_t m, int64_t n, int64_t r);
int launch_project_step_tc(const StepArgs& a, cudaStream_t st) { return launch_project_step_simt(a, st); }
size_t tc_workspace_bytes(int64_t m, int64_t n, int64_t r) { return simt_workspace_bytes(m, n, r); }
size_t refresh_workspace_bytes(int64_t, int64_t, int64_t) { return 0; }
}
extern "C"
int qgalore_refresh_subspace(const uint16_t*, int64_t, int64_t, int64_t, int64_t, int32_t, int32_t, uint64_t,
                             const qg_qtensor*, float*, const qg_qtensor*, int32_t, float*, void*, size_t, int32_t*,
                             void*) { return QG_UNSUPPORTED_SHAPE; }
