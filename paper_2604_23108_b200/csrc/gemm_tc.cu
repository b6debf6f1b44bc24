// placeholder until the tcgen05 path lands
#include "common.cuh"
namespace mohge {
int32_t launch_tc_grouped(const Dims&, int, const GroupPtrs&, const void*, const void*, void*, void*,
                          const int32_t*, const int32_t*, int, int32_t*, Tile*, int64_t, int32_t*,
                          cudaStream_t) {
  set_error("tensor-core path not built");
  return MOHGE_ERR_UNSUPPORTED;
}
}  // namespace mohge
