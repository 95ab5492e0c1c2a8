// Placeholder translation unit for the tcgen05 forward kernel (filled in by the tensor-core path).
#include "lla_common.cuh"

namespace lla {
bool forward_tensor_supported(const ForwardArgs&) { return false; }
int launch_forward_tensor(const ForwardArgs&) { return LLA_ERR_UNSUPPORTED; }
}  // namespace lla
