// Tensor-core (TMA + tcgen05) decode path -- placeholder until the kernel lands.
#include "slim_internal.h"

int slim_tc_shape_ok(int, int, int, int) { return 0; }
int slim_tc_workers(const slim_ctx*) { return 0; }
cudaError_t slim_tc_make_tmap(const slim_ctx*, slim_cache*) { return cudaErrorNotSupported; }
cudaError_t slim_launch_tc(const slim_ctx*, const slim_cache*, const SlimDecodeParams&, cudaStream_t) {
  return cudaErrorNotSupported;
}
