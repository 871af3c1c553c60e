// Shared-memory-resident persistent kernels (placeholder until the packers land).
#include "wrnn_internal.h"

namespace wrnn {
struct ResidentPack { int dummy; };
int resident_supported(const wrnn_model *, int, std::string *why) { if (why) *why = "not built yet"; return WRNN_ERR_UNSUPPORTED; }
int resident_prepare(wrnn_model *m) { m->err = "not built yet"; return WRNN_ERR_UNSUPPORTED; }
void resident_destroy(wrnn_model *) {}
int resident_launch_info(const wrnn_model *, int, int *, int *, int *, int64_t *) { return WRNN_ERR_UNSUPPORTED; }
int resident_run(wrnn_model *, const StepArgs &, cudaStream_t) { return WRNN_ERR_UNSUPPORTED; }
}  // namespace wrnn
