// tcgen05 tensor-core path (bf16 inputs).
#include "pf_common.cuh"

namespace pf {

bool tc_supported(const Problem&) { return false; }
size_t tc_workspace_bytes(const Problem&) { return 0; }
int tc_forward(const Problem&, void*) { return PF_ERR_UNSUPPORTED; }

}  // namespace pf
