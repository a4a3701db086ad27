#include "common.cuh"
namespace fedattn {
size_t decode_scratch_bytes(int, int, int, int) { return 0; }
cudaError_t launch_decode_bf16(const Context *, const DecodeParams &, cudaStream_t, int64_t *) { return cudaErrorNotSupported; }
}
