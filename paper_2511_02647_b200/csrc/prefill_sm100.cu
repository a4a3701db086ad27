#include "common.cuh"
namespace fedattn {
bool prefill_sm100_supported(const Context *) { return false; }
cudaError_t launch_prefill_sm100(const Context *, const PrefillParams &, cudaStream_t, int64_t *) { return cudaErrorNotSupported; }
}
