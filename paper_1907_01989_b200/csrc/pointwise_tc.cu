// Tensor-core pointwise convolution (placeholder until the tcgen05 kernel lands).
#include "kernels.h"

namespace gi {
bool pointwise_tc_supported(int, int) { return false; }
void pointwise_tc_pack(const float*, const float*, int, int, std::vector<uint8_t>*, LaunchRec*) {}
int launch_pointwise_tc(const LaunchRec&, const Ptrs&, void**, int, void*) { return 1; }
void pointwise_tc_release(void*) {}
}  // namespace gi
