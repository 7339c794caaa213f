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
// (the group-mean indicator's rows).  One thread per slot, 128 slots per CTA.  The CTA's 128 key rows are staged in
// shared memory once, as fp32 and transposed ([d][129]: a thread walks its own column without bank conflicts); two
// window queries of all G heads are staged per step ([2][d][G padded to fours]), so that one key element from shared
// memory meets eight query values (two queries x four heads) in registers.  Per (slot, query) the heads are summed in
// ascending order and the dot products in ascending channel order.
constexpr int WR_SLOTS = 128, WR_KPAD = WR_SLOTS + 1, WR_Q = 2;
template <typename T>
__global__ void __launch_bounds__(WR_SLOTS)
window_ring_grouped_kernel(int G, int kv_heads, int T_len, int d, int w, int B, int cap, float scale, const T* __restrict__ q,
                           int64_t qsb, int64_t qsh, int64_t q_head, int64_t st, const float* __restrict__ lse, int64_t lse_sb,
                           int64_t lse_sh, vatp_cache c) {
  extern __shared__ __align__(16) float wr_smem[];
  const int GP = (G + 3) & ~3;
  float* k_s = wr_smem;                          // [d][WR_KPAD]
  float* q_s = wr_smem + (size_t)d * WR_KPAD;    // [WR_Q][d][GP]  (d is a multiple of four: 16-byte aligned)
  const int u = blockIdx.y, tid = threadIdx.x;
  const int slot0 = blockIdx.x * WR_SLOTS, slot = slot0 + tid;
  const int len = min(T_len, B);
  const int b = u / kv_heads, h = u - b * kv_heads;
  const T* qu = q + (int64_t)b * qsb + (int64_t)h * qsh;
  const float* lu = lse + (int64_t)b * lse_sb + (int64_t)h * lse_sh;
  const T* kbase = static_cast<const T*>(c.k_cache) + (int64_t)u * cap * d;
  const int ps = slot < len ? c.pos[(int64_t)u * cap + slot] : -1;
  const float invG = 1.f / (float)G;
  for (int idx = tid; idx < WR_SLOTS * d; idx += WR_SLOTS) {       // consecutive threads: consecutive elements of a row
    const int sl = idx / d, i = idx - sl * d;
    k_s[i * WR_KPAD + sl] = slot0 + sl < cap ? to_f32(kbase[(int64_t)(slot0 + sl) * d + i]) : 0.f;
  }
  for (int idx = tid; idx < WR_Q * d * GP; idx += WR_SLOTS) q_s[idx] = 0.f;      // the padding heads stay zero
  long long fx = 0;
  for (int r0 = 0; r0 < w; r0 += WR_Q) {
    __syncthreads();
    for (int idx = tid; idx < WR_Q * G * d; idx += WR_SLOTS) {
      const int jj = idx / (G * d), rem = idx - jj * (G * d);
      const int g = rem / d, i = rem - g * d;
      const int j = T_len - w + r0 + jj;
      q_s[(jj * d + i) * GP + g] = (r0 + jj < w && j >= 0) ? to_f32(qu[(int64_t)g * q_head + (int64_t)j * st + i]) : 0.f;
    }
    __syncthreads();
    float p[WR_Q];
    bool live[WR_Q];
#pragma unroll
    for (int jj = 0; jj < WR_Q; ++jj) {
      const int j = T_len - w + r0 + jj;
      p[jj] = 0.f;
      live[jj] = slot < cap && r0 + jj < w && j >= 0 && ps >= 0 && ps <= j;      // causal: the token precedes the query
    }
    if (live[0] || live[1]) {
      for (int g0 = 0; g0 < G; g0 += 4) {
        float a[WR_Q][4];
#pragma unroll
        for (int jj = 0; jj < WR_Q; ++jj) a[jj][0] = a[jj][1] = a[jj][2] = a[jj][3] = 0.f;
#pragma unroll 4
        for (int i = 0; i < d; ++i) {
          const float kv = k_s[i * WR_KPAD + tid];
#pragma unroll
          for (int jj = 0; jj < WR_Q; ++jj) {
            const float4 qv = *reinterpret_cast<const float4*>(&q_s[(jj * d + i) * GP + g0]);
            a[jj][0] = fmaf(qv.x, kv, a[jj][0]);
            a[jj][1] = fmaf(qv.y, kv, a[jj][1]);
            a[jj][2] = fmaf(qv.z, kv, a[jj][2]);
            a[jj][3] = fmaf(qv.w, kv, a[jj][3]);
          }
        }
#pragma unroll
        for (int jj = 0; jj < WR_Q; ++jj) {
          const int j = T_len - w + r0 + jj;
          if (live[jj]) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
              if (g0 + k < G) p[jj] += __expf(a[jj][k] * scale - __ldg(lu + (int64_t)(g0 + k) * T_len + j));
          }
        }
      }
    }
#pragma unroll
    for (int jj = 0; jj < WR_Q; ++jj) {
      const int j = T_len - w + r0 + jj;
      if (r0 + jj < w && slot < cap) {
        const float pj = live[jj] ? p[jj] * invG : 0.f;
        const int rr = ((j % w) + w) % w;
        c.ring[((int64_t)u * w + rr) * cap + slot] = pj;
        fx += prob_to_fixed(pj);
      }
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
  const size_t smem = ((size_t)s.d * WR_KPAD + (size_t)WR_Q * s.d * ((G + 3) & ~3)) * sizeof(float);
  if (smem > 200 * 1024 || (s.d & 3)) return cudaErrorNotSupported;
  cudaError_t e = cudaFuncSetAttribute(window_ring_grouped_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(window_ring_grouped_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
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
