// tc_flow: per-chunk flow builder on tcgen05 (see pf_tc.cu for the pipeline).
#include "pf_common.cuh"
#include "pf_tc.cuh"
#include "pf_tc_prims.cuh"

namespace pf {

bool tc_flow_available() { return false; }
int tc_flow_launch(const Problem&, const TcWs&, int) { return PF_ERR_UNSUPPORTED; }

}  // namespace pf
