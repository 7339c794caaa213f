// Internal declarations shared by the kernels of libvatp (not part of the public C ABI).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "vatp.h"

namespace vatp {

struct Shape {
  int units;           // batch * heads
  int heads;
  int T, d;
  int64_t sb, sh, st;  // element strides of q/k/v
  float scale;
  int window;          // 0 = accumulate over all queries (Eq. 2); >0 = last `window` queries (Eq. 3)
  int norm;            // vatp_norm_kind of the value norm in Eq. 4
};

// Value-row norms (Eq. 4 uses l1; the Ablation Study's variants are l2 and l-infinity).  A row is
// folded element by element into a partial, partials of different lanes are merged, and the merged
// partial is finished: l1 sums |x|, l2 sums x^2 and takes the root, l-infinity takes the largest |x|.
__device__ __forceinline__ float norm_fold(int kind, float part, float x) {
  return kind == VATP_NORM_L1 ? part + fabsf(x) : kind == VATP_NORM_L2 ? fmaf(x, x, part) : fmaxf(part, fabsf(x));
}
__device__ __forceinline__ float norm_merge(int kind, float a, float b) { return kind == VATP_NORM_LINF ? fmaxf(a, b) : a + b; }
__device__ __forceinline__ float norm_finish(int kind, float part) { return kind == VATP_NORM_L2 ? sqrtf(part) : part; }

// slots per unit in the decode state: budget + 1, rounded up to a multiple of 8 so that every
// per-slot array of a unit starts on a 32-byte boundary (bulk copies need 16)
__host__ __device__ inline int cache_capacity(int budget) { return (budget + 1 + 7) & ~7; }

// offset (in elements) of unit u's first row
__host__ __device__ inline int64_t unit_offset(const Shape& s, int u) {
  return (int64_t)(u / s.heads) * s.sb + (int64_t)(u % s.heads) * s.sh;
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

// true when the tensor-core kernels are usable on the current device (sm_100, driver entry points found)
bool vatp_tc_available();
// multiprocessors of the current device (looked up once per device)
int device_sm_count();

// 2-D tensor map over `rows` contiguous rows of 128 bf16: box = 64 columns x box_rows rows, 128-byte
// swizzle, rows beyond the end read as zeros.  False when the driver entry point is missing.
bool make_rows_map_bf16(CUtensorMap* m, const void* base, uint64_t rows, uint32_t box_rows);

// 2-D tensor map over `rows` rows of row_words 32-bit words, row_stride_bytes apart (a multiple of 16); the box
// is one row: for gathers of whole rows by row index.  False when the driver entry point is missing.
bool make_row_gather_map(CUtensorMap* m, const void* base, uint32_t row_words, uint64_t rows, uint64_t row_stride_bytes);

// Launch configuration of a kernel that may be scheduled before the previous launch in the stream has
// drained (programmatic dependent launch).  Such a kernel executes griddepcontrol.wait before it reads
// anything an earlier launch wrote.
struct DependentLaunch {
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  DependentLaunch(dim3 grid, dim3 block, size_t smem, cudaStream_t st) : cfg{} {
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
};

// ---- launchers (each returns cudaGetLastError()) ----
// lse_given: `lse` already holds the row normalisers (natural log), pass 1 is skipped
cudaError_t launch_prefill_simt(const Shape& s, int dtype, const void* q, const void* k, const void* v, float* lse,
                                float* attn_acc, float* vnorm, float* score, float* win_rows, cudaStream_t st,
                                bool lse_given = false);
// lse_in: row normalisers [units][T] (natural log) from the caller; non-null skips pass 1
cudaError_t launch_prefill_tc(const Shape& s, const void* q, const void* k, const void* v, float* lse_ws,
                              float* lse_out, float* attn_acc, float* vnorm, float* score, float* win_rows,
                              int32_t* dev_status, cudaStream_t st, const float* lse_in = nullptr);
size_t prefill_tc_workspace_bytes(int units, int T);  // padded log2-domain row normalisers
cudaError_t launch_select(int units, int T, int B, int F, int R, const float* score, int32_t* kept, cudaStream_t st);
cudaError_t launch_compact(const Shape& s, int dtype, int B, const void* k, const void* v, const float* attn_acc,
                           const float* vnorm, const float* win_rows, const int32_t* kept, const vatp_cache& c,
                           int32_t* dev_status, cudaStream_t st);
cudaError_t launch_decode(const Shape& s, int dtype, int B, int F, int R, const vatp_cache& c, const void* q,
                          const void* k, const void* v, void* out, int32_t* evicted, int32_t* dev_status, cudaStream_t st,
                          bool may_overlap);

// bf16, head_dim 128 only; cudaErrorNotSupported when the shape does not fit (take launch_decode's general kernel)
// may_overlap: the caller opted in to launches that run beside earlier decode launches on the stream when they share
// no buffer with them (VATP_FLAG_DECODE_OVERLAP)
cudaError_t launch_decode_mma(const Shape& s, int B, int F, int R, const vatp_cache& c, const void* q, const void* k,
                              const void* v, void* out, int32_t* evicted, int32_t* dev_status, cudaStream_t st,
                              bool may_overlap);
// other work of this library was enqueued on the stream: the next decode launch waits for all of it
// (probe_only: `st` is only a key of the host-side self-test, not a stream the runtime may be asked about)
void decode_history_forget(cudaStream_t st, bool probe_only = false);

bool decode_overlap_policy_probe(void* stream, const uint64_t* begin, const uint64_t* bytes, int n, double share);

// fixed-point image of a probability for the exact window sums (Eq. 3): p in [0, 1] -> p * 2^52
__host__ __device__ inline long long prob_to_fixed(float p) { return (long long)((double)p * 4503599627370496.0); }
__host__ __device__ inline float fixed_to_prob(long long x) { return (float)((double)x * (1.0 / 4503599627370496.0)); }

}  // namespace vatp
