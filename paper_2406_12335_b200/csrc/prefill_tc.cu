// placeholder until the tcgen05 kernel lands
#include "vatp_internal.cuh"
namespace vatp {
bool vatp_tc_available() { return false; }
cudaError_t launch_prefill_tc(const Shape&, const void*, const void*, const void*, float*, float*, float*, float*,
                              float*, int32_t*, cudaStream_t) { return cudaErrorNotSupported; }
}
