// Tensor-core kernel family (placeholder until the tcgen05 kernels land).
#include "dig_common.cuh"
namespace dig {
bool tensor_supports(int, int, int, int, bool) { return false; }
dig_status tensor_gla_fwd(const GlaArgs &) { return DIG_ERR_UNSUPPORTED; }
dig_status tensor_gla_bwd(const GlaArgs &) { return DIG_ERR_UNSUPPORTED; }
}  // namespace dig
