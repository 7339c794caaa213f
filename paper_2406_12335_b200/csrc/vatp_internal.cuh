// Internal declarations shared by the kernels of libvatp (not part of the public C ABI).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "vatp.h"

namespace vatp {

struct Shape {
  int units;           // batch * heads
  int heads;
  int kv_heads;        // 0: k and v have `heads` heads; else grouped queries in ONE launch: the units are the query heads,
                       // k and v have kv_heads heads and unit (b, h) reads KV head h / (heads / kv_heads) of batch b
  int T, d;
  int64_t sb, sh, st;  // element strides of k and v (and of q, unless qsb / qsh say otherwise)
  int64_t qsb, qsh;    // batch and head strides of q (grouped-query attention runs one query head of every KV
                       // group per launch: the units are then the KV heads and q is a strided view)
  int64_t lse_sb, lse_sh;  // where unit (b, h)'s row normalisers start in the caller's [.., T] array: b * lse_sb + h * lse_sh
  int64_t osb, osh;        // likewise for the rows of the attention output [.., T, d] (elements): b * osb + h * osh
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

// Bounds-checking build (-DVATP_DEBUG_BOUNDS): VATP_INB(i, n, status) is false, and records VATP_ERR_BOUNDS in the
// status word, when index i lies outside [0, n); the caller then skips the access.  In the ordinary build it is the
// constant true and costs nothing.
#ifdef VATP_DEBUG_BOUNDS
__device__ __forceinline__ bool vatp_in_bounds(long long i, long long n, int32_t* status) {
  if (i >= 0 && i < n) return true;
  if (status) atomicExch(status, (int)VATP_ERR_BOUNDS);
  return false;
}
#define VATP_INB(i, n, status) vatp::vatp_in_bounds((long long)(i), (long long)(n), (status))
#else
#define VATP_INB(i, n, status) true
#endif

// slots per unit in the decode state: budget + 1, rounded up to a multiple of 8 so that every
// per-slot array of a unit starts on a 32-byte boundary (bulk copies need 16)
__host__ __device__ inline int cache_capacity(int budget) { return (budget + 1 + 7) & ~7; }

// offset (in elements) of unit u's first row in k and v, in q, and in the caller's row-normaliser array
__host__ __device__ inline int64_t unit_offset(const Shape& s, int u) {
  return (int64_t)(u / s.heads) * s.sb + (int64_t)(u % s.heads) * s.sh;
}
__host__ __device__ inline int64_t unit_offset_q(const Shape& s, int u) {
  return (int64_t)(u / s.heads) * s.qsb + (int64_t)(u % s.heads) * s.qsh;
}
__host__ __device__ inline int64_t unit_offset_lse(const Shape& s, int u) {
  return (int64_t)(u / s.heads) * s.lse_sb + (int64_t)(u % s.heads) * s.lse_sh;
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
// attn_out: non-null replaces pass 1 by the fused attention forward, which also writes the output rows (bf16; unit
// (b, h) at b * osb + h * osh, rows of 128 elements)
cudaError_t launch_prefill_tc(const Shape& s, const void* q, const void* k, const void* v, float* lse_ws,
                              float* lse_out, float* attn_acc, float* vnorm, float* score, float* win_rows,
                              int32_t* dev_status, cudaStream_t st, const float* lse_in = nullptr, void* attn_out = nullptr);
// attention forward of the general path: out (unit (b, h) at b * osb + h * osh, rows of d elements) and natural-log normalisers
cudaError_t launch_attention_fwd_general(const Shape& s, int dtype, const void* q, const void* k, const void* v, void* out,
                                         float* lse, cudaStream_t st);
size_t prefill_tc_workspace_bytes(int units, int T);  // padded log2-domain row normalisers
cudaError_t launch_select(int units, int T, int B, int F, int R, const float* score, int32_t* kept, int32_t* dev_status,
                          cudaStream_t st);
cudaError_t launch_compact(const Shape& s, int dtype, int B, const void* k, const void* v, const float* attn_acc,
                           const float* vnorm, const float* win_rows, const int32_t* kept, const vatp_cache& c,
                           int32_t* dev_status, cudaStream_t st);
// windowed decode state from Q, the compacted keys and the row normalisers (natural log): ring, acc_fixed, acc
cudaError_t launch_window_ring_grouped(const Shape& s, int G, int dtype, int B, const void* q, const float* lse, const vatp_cache& c,
                                       cudaStream_t st);
cudaError_t launch_window_ring(const Shape& s, int dtype, int B, const void* q, const float* lse, const vatp_cache& c,
                               int32_t* dev_status, cudaStream_t st);
cudaError_t launch_window_ring_tc(const Shape& s, int B, const void* q, const float* lse, const vatp_cache& c,
                                  int32_t* dev_status, cudaStream_t st);   // bf16, head_dim 128, tensor cores
// grouped-query attention: mean over the group's G partial indicators [G][n] and Eq. 4; the decode step of a KV group
cudaError_t launch_group_mean(int G, int64_t n, const float* part, const float* vnorm, float* attn_acc, float* score,
                              cudaStream_t st);
cudaError_t launch_decode_gqa(int units, int G, int d, int dtype, int B, int F, int R, int window, int norm, float scale,
                              const vatp_cache& c, const void* q, const void* k, const void* v, void* out, int32_t* evicted,
                              int32_t* dev_status, cudaStream_t st);
cudaError_t launch_decode(const Shape& s, int dtype, int B, int F, int R, const vatp_cache& c, const void* q,
                          const void* k, const void* v, void* out, int32_t* evicted, int32_t* dev_status, cudaStream_t st,
                          bool may_overlap);

// bf16, head_dim 128 only; cudaErrorNotSupported when the shape does not fit (take launch_decode's general kernel)
// may_overlap: the caller opted in to launches that run beside earlier decode launches on the stream when they share
// no buffer with them (VATP_FLAG_DECODE_OVERLAP)
// G: query heads per cache (grouped-query attention, 1 .. 8): s.units counts caches, q and out hold G rows per unit
cudaError_t launch_decode_mma(const Shape& s, int B, int F, int R, const vatp_cache& c, const void* q, const void* k,
                              const void* v, void* out, int32_t* evicted, int32_t* dev_status, cudaStream_t st,
                              bool may_overlap, int G = 1);
// other work of this library was enqueued on the stream: the next decode launch waits for all of it
// (probe_only: `st` is only a key of the host-side self-test, not a stream the runtime may be asked about)
void decode_history_forget(cudaStream_t st, bool probe_only = false);

bool decode_overlap_policy_probe(void* stream, const uint64_t* begin, const uint64_t* bytes, int n, double share);

// Fixed-point image of a probability for the exact window sums (Eq. 3): p in [0, 1] -> trunc(p * 2^52), taken from
// the bits of the float: its 24-bit significand shifted by (biased exponent - 98).  Exact, like the product in
// double precision it replaces, without the conversions (which run at a fraction of the integer rate).
__host__ __device__ inline long long prob_to_fixed(float p) {
#ifdef __CUDA_ARCH__
  // on the device the same value in two instructions: the product with 2^52 is exact in fp32 (a power of two), and
  // the conversion truncates towards zero (negative or NaN inputs do not occur: p is a probability)
  return __float2ll_rz(p * 4503599627370496.0f);
#else
  uint32_t b;
  memcpy(&b, &p, sizeof(b));
  const int e = (int)((b >> 23) & 0xffu);
  if (e == 0 || (b >> 31)) return 0;                   // zero, subnormal (below 2^-52 in any case) or negative
  const long long m = (long long)((b & 0x7fffffu) | 0x800000u);
  const int s = e - 98;                                // p = m * 2^(e - 150); times 2^52
  return s >= 0 ? (s < 39 ? m << s : 0x7fffffffffffffffll) : (s > -24 ? m >> -s : 0);
#endif
}
__host__ __device__ inline float fixed_to_prob(long long x) { return (float)((double)x * (1.0 / 4503599627370496.0)); }

}  // namespace vatp
