// placeholder until the MoE path lands
#include "qmm_common.cuh"
namespace qmm {
size_t moe_workspace_bytes(const qmm_moe_args*) { return 256; }
qmm_status launch_moe(const qmm_moe_args*, void*, bool, cudaStream_t) { return fail(QMM_ERR_UNSUPPORTED, "qmm_moe: not built yet"); }
}
