// Placeholders for entry points whose kernels are not written yet.
#include "qg_common.cuh"
namespace qg {
size_t refresh_workspace_bytes(int64_t, int64_t, int64_t) { return 0; }
}
extern "C"
int qgalore_refresh_subspace(const uint16_t*, int64_t, int64_t, int64_t, int64_t, int32_t, int32_t, uint64_t,
                             const qg_qtensor*, float*, const qg_qtensor*, int32_t, float*, void*, size_t, int32_t*,
                             void*) { return QG_UNSUPPORTED_SHAPE; }
