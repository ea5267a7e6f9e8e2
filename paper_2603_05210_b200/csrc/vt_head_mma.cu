// Draft head, tensor-core path (placeholder until the tcgen05 kernel lands).
#include "vt_launch.h"

namespace vt {
vt_status launch_head_mma(const HeadCall&, cudaStream_t) { return VT_ERR_UNSUPPORTED; }
}  // namespace vt
