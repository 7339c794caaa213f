// History-window state of the decode step (Eq. 3) rebuilt from Q and the compacted keys.
//
// The windowed indicator needs, per kept token, its probability under each of the last w prompt queries:
// ring[u][j mod w][slot] = a_slot^j for j = T - w .. T - 1, and the exact fixed-point sum of those w values
// (the indicator itself).  Rather than have the scoring pass write all w x T probabilities of a unit and
// gather B + 1 of their columns afterwards, this kernel recomputes the w x cap block that is kept:
//   p[j][slot] = exp(scale * <q_j, k_slot> - lse_j)   for pos[slot] <= j (causal), else 0
// a w x cap x d contraction per unit (tiny next to the T x T scoring passes), written straight into the ring's
// layout.  bf16 with head_dim 128 runs on the tensor cores (window_ring_tc_kernel, beside the scoring kernel whose
// machinery it shares); this file holds the dispatch and the general kernel.  The sums are integers (2^52 fixed
// point), so they do not depend on the order in which rows are added.
#include "vatp_internal.cuh"

namespace vatp {
namespace {

// Any dtype / head_dim: one thread per slot, FMA dot products (small shapes and fp32 inputs).
template <typename T>
__global__ void __launch_bounds__(128)
window_ring_general_kernel(int heads, int T_len, int d, int w, int B, int cap, float scale, const T* __restrict__ q,
                           int64_t sb, int64_t sh, int64_t st, const float* __restrict__ lse, vatp_cache c) {
  extern __shared__ float q_row[];       // the current query row, fp32
  const int u = blockIdx.y;
  const int slot = blockIdx.x * blockDim.x + threadIdx.x;
  const int len = min(T_len, B);
  const T* qu = q + (int64_t)(u / heads) * sb + (int64_t)(u % heads) * sh;
  const T* krow = static_cast<const T*>(c.k_cache) + ((int64_t)u * cap + slot) * d;
  const int ps = slot < len ? c.pos[(int64_t)u * cap + slot] : -1;
  long long fx = 0;
  for (int r = 0; r < w; ++r) {
    const int j = T_len - w + r;
    const int rr = ((j % w) + w) % w;
    __syncthreads();
    if (j >= 0)
      for (int i = threadIdx.x; i < d; i += blockDim.x) q_row[i] = to_f32(qu[(int64_t)j * st + i]);
    __syncthreads();
    float p = 0.f;
    if (slot < cap && j >= 0 && ps >= 0 && ps <= j) {
      float dot = 0.f;
      for (int i = 0; i < d; ++i) dot = fmaf(q_row[i], to_f32(krow[i]), dot);
      p = __expf(dot * scale - __ldg(lse + (int64_t)u * T_len + j));
    }
    if (slot < cap) {
      c.ring[((int64_t)u * w + rr) * cap + slot] = p;
      fx += prob_to_fixed(p);
    }
  }
  if (slot < cap) {
    c.acc_fixed[(int64_t)u * cap + slot] = fx;
    c.acc[(int64_t)u * cap + slot] = fixed_to_prob(fx);
  }
}

// Grouped-query attention: the history holds the MEAN over the KV group's G query heads of their probabilities
// (the group-mean indicator's rows).  A plain kernel like the one above: one thread per slot, the G query rows of
// the current position in shared memory, heads summed in ascending order.
template <typename T>
__global__ void __launch_bounds__(128)
window_ring_grouped_kernel(int G, int kv_heads, int T_len, int d, int w, int B, int cap, float scale, const T* __restrict__ q,
                           int64_t qsb, int64_t qsh, int64_t q_head, int64_t st, const float* __restrict__ lse, int64_t lse_sb,
                           int64_t lse_sh, vatp_cache c) {
  extern __shared__ float q_rows[];      // [G][d], fp32
  const int u = blockIdx.y;
  const int slot = blockIdx.x * blockDim.x + threadIdx.x;
  const int len = min(T_len, B);
  const int b = u / kv_heads, h = u - b * kv_heads;
  const T* qu = q + (int64_t)b * qsb + (int64_t)h * qsh;
  const float* lu = lse + (int64_t)b * lse_sb + (int64_t)h * lse_sh;
  const T* krow = static_cast<const T*>(c.k_cache) + ((int64_t)u * cap + slot) * d;
  const int ps = slot < len ? c.pos[(int64_t)u * cap + slot] : -1;
  const float invG = 1.f / (float)G;
  long long fx = 0;
  for (int r = 0; r < w; ++r) {
    const int j = T_len - w + r;
    const int rr = ((j % w) + w) % w;
    __syncthreads();
    if (j >= 0)
      for (int i = threadIdx.x; i < G * d; i += blockDim.x)
        q_rows[i] = to_f32(qu[(int64_t)(i / d) * q_head + (int64_t)j * st + (i % d)]);
    __syncthreads();
    float p = 0.f;
    if (slot < cap && j >= 0 && ps >= 0 && ps <= j) {
      for (int g = 0; g < G; ++g) {
        float dot = 0.f;
        for (int i = 0; i < d; ++i) dot = fmaf(q_rows[g * d + i], to_f32(krow[i]), dot);
        p += __expf(dot * scale - __ldg(lu + (int64_t)g * T_len + j));
      }
      p *= invG;
    }
    if (slot < cap) {
      c.ring[((int64_t)u * w + rr) * cap + slot] = p;
      fx += prob_to_fixed(p);
    }
  }
  if (slot < cap) {
    c.acc_fixed[(int64_t)u * cap + slot] = fx;
    c.acc[(int64_t)u * cap + slot] = fixed_to_prob(fx);
  }
}

}  // namespace

// lse: [batch, heads, T] contiguous (every query head's normalisers); s describes the KV units (see make_shape)
cudaError_t launch_window_ring_grouped(const Shape& s, int G, int dtype, int B, const void* q, const float* lse, const vatp_cache& c,
                                       cudaStream_t st) {
  const int cap = cache_capacity(B);
  const size_t smem = (size_t)G * s.d * sizeof(float);
  if (smem > 48 * 1024) return cudaErrorNotSupported;
  const dim3 grid((cap + 127) / 128, s.units);
  if (dtype == VATP_F32)
    window_ring_grouped_kernel<float><<<grid, 128, smem, st>>>(G, s.heads, s.T, s.d, s.window, B, cap, s.scale, static_cast<const float*>(q),
                                                                s.qsb, s.qsh, s.sh, s.st, lse, s.lse_sb, s.lse_sh, c);
  else
    window_ring_grouped_kernel<__nv_bfloat16><<<grid, 128, smem, st>>>(G, s.heads, s.T, s.d, s.window, B, cap, s.scale,
                                                                        static_cast<const __nv_bfloat16*>(q), s.qsb, s.qsh, s.sh, s.st,
                                                                        lse, s.lse_sb, s.lse_sh, c);
  return cudaGetLastError();
}

cudaError_t launch_window_ring(const Shape& s, int dtype, int B, const void* q, const float* lse, const vatp_cache& c,
                               int32_t* dev_status, cudaStream_t st) {
  const int cap = cache_capacity(B);
  if (dtype == VATP_BF16 && s.d == 128 && vatp_tc_available()) return launch_window_ring_tc(s, B, q, lse, c, dev_status, st);
  if (dtype == VATP_F32) {
    window_ring_general_kernel<float><<<dim3((cap + 127) / 128, s.units), 128, s.d * sizeof(float), st>>>(
        s.heads, s.T, s.d, s.window, B, cap, s.scale, static_cast<const float*>(q), s.qsb, s.qsh, s.st, lse, c);
  } else {
    window_ring_general_kernel<__nv_bfloat16><<<dim3((cap + 127) / 128, s.units), 128, s.d * sizeof(float), st>>>(
        s.heads, s.T, s.d, s.window, B, cap, s.scale, static_cast<const __nv_bfloat16*>(q), s.qsb, s.qsh, s.st, lse, c);
  }
  return cudaGetLastError();
}

}  // namespace vatp
