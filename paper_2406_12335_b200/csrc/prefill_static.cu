// Prefill scoring for callers that cannot allocate device memory.
//
// vatp_prefill_scores needs a few hundred kilobytes of device scratch (the row normalisers that
// pass 1 hands to pass 2) and asks the caller for it.  Some callers have nowhere to get it from: a
// plugin running inside a host application that owns the allocator and hands out no scratch, code
// on a latency-critical path where a cudaMalloc (which synchronises the device) is forbidden, or a
// process whose memory pool was sized up front and is full.  For them the scratch lives in a
// file-scope device array that is part of the library image: every GPU that loads the library
// holds VATP_STATIC_SCRATCH_BYTES of it until the process exits, and nothing is allocated or freed
// at call time.
#include <mutex>

#include "vatp_internal.cuh"

namespace {

static __device__ __align__(256) unsigned char g_static_scratch[VATP_STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` names a host-side shadow of the array, not device memory, so the
// device address is looked up once per device (with that device current) and kept here.
constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};
std::mutex g_setup_mutex;

cudaError_t scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" vatp_status vatp_prefill_scores_static(const vatp_params* params, const void* q, const void* k,
                                                  const void* v, float* lse_out, float* attn_acc, float* vnorm,
                                                  float* score, float* win_rows, int32_t* dev_status,
                                                  void* cuda_stream) {
  if (!params) return VATP_ERR_INVALID_ARG;
  const size_t need = vatp_workspace_bytes(params);   // 0 when the parameters are invalid
  if (need > VATP_STATIC_SCRATCH_BYTES) return VATP_ERR_STATIC_SCRATCH;
  void* scratch = nullptr;
  if (need > 0 && scratch_address(&scratch) != cudaSuccess) return VATP_ERR_CUDA;
  // Nothing in the scratch has to start at zero: pass 1 writes every normaliser that pass 2 reads.
  // Two calls on one stream do not race on the array although pass 2 lets the work after it start early:
  // every call begins by zeroing its work-item counters, either with an ordinary (fully serialising)
  // cudaMemsetAsync or with a one-warp kernel that executes griddepcontrol.wait first, and the kernel after it
  // (pass 1, resident early as that kernel's programmatic dependent) also waits before it touches global memory:
  // both waits return only when everything earlier in the stream, the previous call's pass 2 included, has completed.
  // With invalid parameters (need == 0) the call below reports the precise reason.
  return vatp_prefill_scores(params, q, k, v, lse_out, attn_acc, vnorm, score, win_rows, scratch,
                             VATP_STATIC_SCRATCH_BYTES, dev_status, cuda_stream);
}
