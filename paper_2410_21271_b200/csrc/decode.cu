// Decode kernel family (M <= 64).
#include "eora_common.cuh"
namespace eora {
bool decode_supported(const Handle*, int) { return false; }
void decode_make_plan(Handle* h) { h->plan = DecodePlan(); }
cudaError_t launch_decode_forward(const Handle*, const void*, int, void*, cudaStream_t) { return cudaErrorNotSupported; }
int decode_launch_count(const Handle*, int) { return 1; }
}  // namespace eora
