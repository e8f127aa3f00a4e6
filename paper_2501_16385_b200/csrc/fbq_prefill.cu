// Prefill kernel (M > 16) of the FBQuant linear -- placeholder until the
// tcgen05 / TMEM kernel lands: reports "not supported" so that the dispatcher
// routes large-M calls to the generic kernel.
#include "fbq_common.cuh"

namespace fbq {

bool prefill_supported(const LinearArgs &) { return false; }

cudaError_t launch_prefill(const LinearArgs &, Workspace &, cudaStream_t, int *)
{
    return cudaErrorInvalidConfiguration;
}

}  // namespace fbq
