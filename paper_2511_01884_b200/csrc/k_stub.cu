// placeholder planners for kernel families that are not written yet
#include "plan.h"
namespace forge {
#define STUB(n) \
forge_status_t n##_plan(const forge_fused_linear_desc_t &, int, forge_plan_info_t *, WorkspaceLayout *) { return FORGE_ERR_UNSUPPORTED; } \
forge_status_t n##_setup(Handle &) { return FORGE_ERR_UNSUPPORTED; } \
forge_status_t n##_launch(Handle &, const RunArgs &) { return FORGE_ERR_UNSUPPORTED; }
STUB(k3) STUB(k4)
}
