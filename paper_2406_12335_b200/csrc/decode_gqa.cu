// Decode step for grouped-query attention: the G query heads of a KV group attend over ONE shared, budgeted
// cache.  The paper leaves this case to future work ("Compatibility with grouped-query attention") and points
// at a group-wise score; here the indicator of a cached token advances by the MEAN of the probabilities the
// group's heads give it (Eq. 2 under that mean; with a history window, Eq. 3: that mean row enters the ring
// and the exact fixed-point window sum moves by it), Eq. 4 multiplies by the norm of the shared value row, and
// the lowest importance is released as in the multi-head step.
//
// A plain kernel, not a tuned one: one CTA per KV unit, any dtype and head_dim, the logits of all heads
// in shared memory.  Steps: append (k, v); per head logits, max, sum; per head output; indicator update and
// arg-min over the slots.
#include "vatp_internal.cuh"

namespace vatp {
namespace {

constexpr int GQ_THREADS = 256;

__device__ __forceinline__ float block_max(float x, float* red) {
#pragma unroll
  for (int o = 16; o; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
  __syncthreads();
  float y = red[0];
  for (int i = 1; i < GQ_THREADS / 32; ++i) y = fmaxf(y, red[i]);
  return y;
}
__device__ __forceinline__ float block_sum(float x, float* red) {
#pragma unroll
  for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
  __syncthreads();
  float y = 0.f;
  for (int i = 0; i < GQ_THREADS / 32; ++i) y += red[i];      // fixed order
  return y;
}

template <typename T>
__global__ void __launch_bounds__(GQ_THREADS)
decode_gqa_kernel(int G, int d, int B, int cap, int F, int R, int w, int norm, float scale, vatp_cache c, const T* __restrict__ q_new,
                  const T* __restrict__ k_new, const T* __restrict__ v_new, T* __restrict__ out, int32_t* __restrict__ evicted,
                  int32_t* dev_status) {
  extern __shared__ float gq_smem[];            // p[G][cap] (logits, then probabilities) | q[G][d]
  __shared__ float red[GQ_THREADS / 32];
  __shared__ unsigned long long key_red[GQ_THREADS / 32];
  __shared__ int slot_red[GQ_THREADS / 32], pos_red[GQ_THREADS / 32];
  float* p_s = gq_smem;
  float* q_s = gq_smem + (size_t)G * cap;
  const int u = blockIdx.x, tid = threadIdx.x;
  const int len = c.len[u], fs = c.free_slot[u], t = c.next_pos[u];
  if (!VATP_INB(len, cap, dev_status) || !VATP_INB(fs, cap, dev_status)) return;
  const int hi = len + 1;
  T* kc = static_cast<T*>(c.k_cache) + (int64_t)u * cap * d;
  T* vc = static_cast<T*>(c.v_cache) + (int64_t)u * cap * d;

  // ---- append the new token (Eq. 4: its norm) and stage the group's queries
  float nn = 0.f;
  for (int i = tid; i < d; i += GQ_THREADS) {
    kc[(int64_t)fs * d + i] = k_new[(int64_t)u * d + i];
    const T x = v_new[(int64_t)u * d + i];
    vc[(int64_t)fs * d + i] = x;
    nn = norm_fold(norm, nn, to_f32(x));
  }
  for (int i = tid; i < G * d; i += GQ_THREADS) q_s[i] = to_f32(q_new[(int64_t)u * G * d + i]);
  // the norm's partials are merged in a fixed order
  {
#pragma unroll
    for (int o = 16; o; o >>= 1) nn = norm_merge(norm, nn, __shfl_xor_sync(0xffffffffu, nn, o));
    __syncthreads();
    if ((tid & 31) == 0) red[tid >> 5] = nn;
    __syncthreads();
    nn = red[0];
    for (int i = 1; i < GQ_THREADS / 32; ++i) nn = norm_merge(norm, nn, red[i]);
    nn = norm_finish(norm, nn);
  }
  __syncthreads();                              // the appended rows and the queries are visible to the CTA

  // ---- logits of every head over the live slots
  for (int s = tid; s < hi; s += GQ_THREADS) {
    const T* kr = kc + (int64_t)s * d;
    for (int g = 0; g < G; ++g) {
      float dot = 0.f;
      for (int i = 0; i < d; ++i) dot = fmaf(q_s[g * d + i], to_f32(kr[i]), dot);
      p_s[(size_t)g * cap + s] = dot * scale;
    }
  }
  __syncthreads();
  // ---- per head: softmax over the slots, then the output row (Eq. 1)
  for (int g = 0; g < G; ++g) {
    float m = -INFINITY;
    for (int s = tid; s < hi; s += GQ_THREADS) m = fmaxf(m, p_s[(size_t)g * cap + s]);
    m = block_max(m, red);
    float l = 0.f;
    for (int s = tid; s < hi; s += GQ_THREADS) {
      const float e = __expf(p_s[(size_t)g * cap + s] - m);
      p_s[(size_t)g * cap + s] = e;
      l += e;
    }
    l = block_sum(l, red);
    const float inv = 1.f / l;
    for (int s = tid; s < hi; s += GQ_THREADS) p_s[(size_t)g * cap + s] *= inv;
    __syncthreads();
    for (int i = tid; i < d; i += GQ_THREADS) {
      float a = 0.f;
      for (int s = 0; s < hi; ++s) a = fmaf(p_s[(size_t)g * cap + s], to_f32(vc[(int64_t)s * d + i]), a);
      if constexpr (sizeof(T) == 2) out[((int64_t)u * G + g) * d + i] = __float2bfloat16(a);
      else out[((int64_t)u * G + g) * d + i] = a;
    }
  }
  __syncthreads();
  // ---- indicator += mean of the heads' probabilities; importance; arg-min among the unprotected slots
  const bool evicting = hi > B;
  unsigned long long my_key = ~0ull;
  int my_slot = -1, my_pos = -1;
  const float invG = 1.f / (float)G;
  for (int s = tid; s < hi; s += GQ_THREADS) {
    float pm = 0.f;
    for (int g = 0; g < G; ++g) pm += p_s[(size_t)g * cap + s];
    pm *= invG;
    const int64_t o = (int64_t)u * cap + s;
    const bool is_new = s == fs;
    float S;
    if (w > 0) {
      // Eq. 3: row t mod w of the ring is replaced; the window sum is kept as an exact integer
      float* ring_row = c.ring + ((int64_t)u * w + (t % w)) * cap;
      const long long fx = is_new ? prob_to_fixed(pm) : c.acc_fixed[o] + prob_to_fixed(pm) - prob_to_fixed(ring_row[s]);
      ring_row[s] = pm;
      c.acc_fixed[o] = fx;
      S = fixed_to_prob(fx);
    } else {
      S = is_new ? pm : c.acc[o] + pm;
    }
    c.acc[o] = S;
    if (is_new) { c.vnorm[o] = nn; c.pos[o] = t; }
    if (evicting) {
      const int ps = is_new ? t : c.pos[o];
      const float I = S * (is_new ? nn : c.vnorm[o]);
      if (ps >= F && ps <= t - R) {
        const unsigned long long key = ((unsigned long long)__float_as_uint(I) << 32) | (unsigned)(0x7fffffff - ps);
        if (key < my_key) { my_key = key; my_slot = s; my_pos = ps; }
      }
    }
  }
  // recycled slot: the other rows of its ring column belong to the previous occupant
  for (int rr = tid; rr < w; rr += GQ_THREADS)
    if (rr != t % w) c.ring[((int64_t)u * w + rr) * cap + fs] = 0.f;
  if (!evicting) {
    if (tid == 0) {
      c.len[u] = hi; c.free_slot[u] = hi; c.next_pos[u] = t + 1; c.last_slot[u] = fs;
      if (evicted) evicted[u] = -1;
    }
    return;
  }
  // lowest key of the CTA: warps first, then warp 0 over the warps' candidates
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    const unsigned long long k2 = __shfl_xor_sync(0xffffffffu, my_key, o);
    const int s2 = __shfl_xor_sync(0xffffffffu, my_slot, o), p2 = __shfl_xor_sync(0xffffffffu, my_pos, o);
    if (k2 < my_key) { my_key = k2; my_slot = s2; my_pos = p2; }
  }
  if ((tid & 31) == 0) { key_red[tid >> 5] = my_key; slot_red[tid >> 5] = my_slot; pos_red[tid >> 5] = my_pos; }
  __syncthreads();
  if (tid == 0) {
    unsigned long long best = ~0ull;
    int bs = -1, bp = -1;
    for (int i = 0; i < GQ_THREADS / 32; ++i)
      if (key_red[i] < best) { best = key_red[i]; bs = slot_red[i]; bp = pos_red[i]; }
    if (bs >= 0) {
      c.pos[(int64_t)u * cap + bs] = -1;
      c.free_slot[u] = bs;
      c.len[u] = hi - 1;
      if (evicted) evicted[u] = bp;
    } else {
      c.len[u] = hi;
      c.free_slot[u] = min(hi, cap - 1);
      if (evicted) evicted[u] = -1;
    }
    c.next_pos[u] = t + 1;
    c.last_slot[u] = fs;
  }
}

// attn_acc[u][t] = mean over the group's G partial indicators; score = that mean times the value norm (Eq. 4)
__global__ void group_mean_kernel(int G, int64_t n, const float* __restrict__ part, const float* __restrict__ vnorm,
                                  float* __restrict__ attn_acc, float* __restrict__ score) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float s = 0.f;
  for (int g = 0; g < G; ++g) s += part[(int64_t)g * n + i];       // fixed order
  s *= 1.f / (float)G;
  attn_acc[i] = s;
  score[i] = s * vnorm[i];
}

}  // namespace

cudaError_t launch_group_mean(int G, int64_t n, const float* part, const float* vnorm, float* attn_acc, float* score,
                              cudaStream_t st) {
  group_mean_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(G, n, part, vnorm, attn_acc, score);
  return cudaGetLastError();
}

// units: batch * kv_heads.  cudaErrorNotSupported when the logits of a unit's heads do not fit in shared memory.
cudaError_t launch_decode_gqa(int units, int G, int d, int dtype, int B, int F, int R, int window, int norm, float scale,
                              const vatp_cache& c, const void* q, const void* k, const void* v, void* out, int32_t* evicted,
                              int32_t* dev_status, cudaStream_t st) {
  const int cap = cache_capacity(B);
  const size_t smem = sizeof(float) * ((size_t)G * cap + (size_t)G * d);
  if (smem > 200 * 1024) return cudaErrorNotSupported;
  cudaError_t e;
  if (dtype == VATP_F32) {
    e = cudaFuncSetAttribute(decode_gqa_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    decode_gqa_kernel<float><<<units, GQ_THREADS, smem, st>>>(G, d, B, cap, F, R, window, norm, scale, c, (const float*)q, (const float*)k,
                                                               (const float*)v, (float*)out, evicted, dev_status);
  } else {
    e = cudaFuncSetAttribute(decode_gqa_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    decode_gqa_kernel<__nv_bfloat16><<<units, GQ_THREADS, smem, st>>>(G, d, B, cap, F, R, window, norm, scale, c, (const __nv_bfloat16*)q,
                                                                        (const __nv_bfloat16*)k, (const __nv_bfloat16*)v,
                                                                        (__nv_bfloat16*)out, evicted, dev_status);
  }
  return cudaGetLastError();
}

}  // namespace vatp
