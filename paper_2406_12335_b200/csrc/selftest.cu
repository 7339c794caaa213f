// Self-test of the bounded device-side wait that every pipeline of this library uses: one CTA waits
// on a shared-memory barrier that nothing ever arms, gives up after `limit_ns`, reports
// VATP_ERR_TIMEOUT through the status word and returns normally - no trap, no endless loop, the
// context stays usable.
#include "vatp_internal.cuh"

namespace {

__device__ __forceinline__ bool try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(parity) : "memory");
  return ok != 0;
}

__global__ void bounded_wait_kernel(unsigned long long limit_ns, int32_t* dev_status, unsigned long long* waited_ns) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(&bar)), "r"(1) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t0, t1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    bool done = false;
    do {
      done = try_wait(&bar, 0);          // phase 0 never completes: nobody arrives
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
    } while (!done && t1 - t0 <= limit_ns);
    if (!done && dev_status) atomicExch(dev_status, (int)VATP_ERR_TIMEOUT);
    if (waited_ns) *waited_ns = t1 - t0;
  }
}

}  // namespace

extern "C" int32_t vatp_selftest_overlap_policy(void* stream, const uint64_t* begin, const uint64_t* bytes, int32_t n,
                                                double share) {
  if (share < 0.0) {        // what any other call of the library on the stream does to the record
    vatp::decode_history_forget(static_cast<cudaStream_t>(stream), true);
    return 0;
  }
  if (!begin || !bytes || n <= 0) return -1;
  return vatp::decode_overlap_policy_probe(stream, begin, bytes, n, share) ? 1 : 0;
}

extern "C" vatp_status vatp_selftest_bounded_wait(uint64_t limit_ns, int32_t* dev_status, uint64_t* waited_ns,
                                                  void* cuda_stream) {
  if (!dev_status) return VATP_ERR_INVALID_ARG;
  if (limit_ns == 0 || limit_ns > 100000000ull) return VATP_ERR_INVALID_ARG;   // at most 0.1 s
  bounded_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      limit_ns, dev_status, reinterpret_cast<unsigned long long*>(waited_ns));
  return cudaGetLastError() == cudaSuccess ? VATP_OK : VATP_ERR_CUDA;
}
