// Placeholder until the tcgen05 forward kernel lands: no shape is claimed by the fast path.
#include "rib_common.cuh"
namespace rib {
bool sm100_fwd_supported(const Problem&) { return false; }
cudaError_t sm100_fwd(const Problem&, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace rib
