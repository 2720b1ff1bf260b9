// sm_100a tensor-core path (placeholder until the tcgen05 kernels land).
#include "rglru_internal.h"

namespace rglru {
bool sm100_prefill_supported(int, int, int, int, int) { return false; }
size_t sm100_prefill_workspace_bytes(int, int, int, int) { return 0; }
cudaError_t sm100_prefill(const FwdArgs &, void *, size_t, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace rglru
