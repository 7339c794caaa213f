// Attention forward for shapes the tensor-core kernel does not take (any dtype, head_dim <= 256): the layer's
// output rows out[j] = sum_{i<=j} a_i^j v_i (Section 3.1, Eq. 1) and the row normalisers lse[j], which the
// scoring pass then reuses instead of recomputing them.
// A plain kernel for small shapes: one warp per query row walks the keys 0..j in order with a running
// maximum, sum and output (lane c holds channels c, c + 32, ...); the dot product is reduced over the warp.
#include "vatp_internal.cuh"

namespace vatp {
namespace {

constexpr int FG_WARPS = 4;
constexpr int FG_MAXC = 8;       // channels per lane: head_dim <= 256

template <typename T>
__global__ void __launch_bounds__(FG_WARPS * 32)
attention_fwd_general_kernel(int heads, int T_len, int d, float scale, const T* __restrict__ q, const T* __restrict__ k,
                             const T* __restrict__ v, int64_t sb, int64_t sh, int64_t st, int64_t qsb, int64_t qsh,
                             T* __restrict__ out, int64_t osb, int64_t osh, float* __restrict__ lse, int64_t lse_sb, int64_t lse_sh) {
  const int u = blockIdx.y, lane = threadIdx.x & 31;
  const int j = blockIdx.x * FG_WARPS + (threadIdx.x >> 5);
  if (j >= T_len) return;
  const int b = u / heads, h = u - b * heads;
  const T* qr = q + (int64_t)b * qsb + (int64_t)h * qsh + (int64_t)j * st;
  const T* ku = k + (int64_t)b * sb + (int64_t)h * sh;
  const T* vu = v + (int64_t)b * sb + (int64_t)h * sh;
  float qv[FG_MAXC], acc[FG_MAXC];
#pragma unroll
  for (int c = 0; c < FG_MAXC; ++c) {
    const int ch = lane + 32 * c;
    qv[c] = ch < d ? to_f32(qr[ch]) : 0.f;
    acc[c] = 0.f;
  }
  float m = -INFINITY, l = 0.f;
  for (int i = 0; i <= j; ++i) {
    const T* kr = ku + (int64_t)i * st;
    const T* vr = vu + (int64_t)i * st;
    float dot = 0.f;
#pragma unroll
    for (int c = 0; c < FG_MAXC; ++c) {
      const int ch = lane + 32 * c;
      if (ch < d) dot = fmaf(qv[c], to_f32(kr[ch]), dot);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);     // every lane holds the same sum
    const float s = dot * scale;
    if (s > m) {
      const float f = expf(m - s);      // 0 on the first key
      l *= f;
#pragma unroll
      for (int c = 0; c < FG_MAXC; ++c) acc[c] *= f;
      m = s;
    }
    const float p = expf(s - m);
    l += p;
#pragma unroll
    for (int c = 0; c < FG_MAXC; ++c) {
      const int ch = lane + 32 * c;
      if (ch < d) acc[c] = fmaf(p, to_f32(vr[ch]), acc[c]);
    }
  }
  const float inv = 1.f / l;
  T* orow = out + (int64_t)b * osb + (int64_t)h * osh + (int64_t)j * d;
#pragma unroll
  for (int c = 0; c < FG_MAXC; ++c) {
    const int ch = lane + 32 * c;
    if (ch < d) {
      if constexpr (sizeof(T) == 2) orow[ch] = __float2bfloat16(acc[c] * inv);
      else orow[ch] = acc[c] * inv;
    }
  }
  if (lane == 0) lse[(int64_t)b * lse_sb + (int64_t)h * lse_sh + j] = m + logf(l);
}

}  // namespace

// out: the inputs' dtype, unit (b, h)'s rows at b * osb + h * osh; lse: natural log, unit (b, h) at b * lse_sb + h * lse_sh.
cudaError_t launch_attention_fwd_general(const Shape& s, int dtype, const void* q, const void* k, const void* v, void* out,
                                         float* lse, cudaStream_t st) {
  if (s.d > 32 * FG_MAXC) return cudaErrorNotSupported;
  const dim3 grid((s.T + FG_WARPS - 1) / FG_WARPS, s.units);
  if (dtype == VATP_F32)
    attention_fwd_general_kernel<float><<<grid, FG_WARPS * 32, 0, st>>>(
        s.heads, s.T, s.d, s.scale, static_cast<const float*>(q), static_cast<const float*>(k), static_cast<const float*>(v),
        s.sb, s.sh, s.st, s.qsb, s.qsh, static_cast<float*>(out), s.osb, s.osh, lse, s.lse_sb, s.lse_sh);
  else
    attention_fwd_general_kernel<__nv_bfloat16><<<grid, FG_WARPS * 32, 0, st>>>(
        s.heads, s.T, s.d, s.scale, static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k),
        static_cast<const __nv_bfloat16*>(v), s.sb, s.sh, s.st, s.qsb, s.qsh, static_cast<__nv_bfloat16*>(out), s.osb, s.osh, lse,
        s.lse_sb, s.lse_sh);
  return cudaGetLastError();
}

}  // namespace vatp
