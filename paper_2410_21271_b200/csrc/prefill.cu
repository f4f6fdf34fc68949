// Prefill kernel family (large M, tcgen05).
#include "eora_common.cuh"
namespace eora {
bool prefill_supported(const Handle*, int) { return false; }
cudaError_t prefill_init(Handle*) { return cudaSuccess; }
void prefill_free(Handle*) {}
cudaError_t launch_prefill_forward(const Handle*, const void*, int, void*, cudaStream_t) { return cudaErrorNotSupported; }
int prefill_launch_count(const Handle*, int) { return 2; }
}  // namespace eora
