// placeholder while the API is reworked
#include "common.cuh"
namespace im2win {
int launch_conv_tc_strip(const void*, const float*, float*, const Geometry&, int, cudaStream_t, Scratch, int, bool) {
  return IM2WIN_EUNSUPPORTED;
}
size_t strip_scratch_bytes(const Geometry&, int, int) { return 0; }
}  // namespace im2win
