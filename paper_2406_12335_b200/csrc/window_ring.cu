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
// (the group-mean indicator's rows).  A CTA of four warps takes 128 slots: their key rows are staged in shared memory
// once, as fp32 and transposed ([d][132]), and eight window queries of all G heads per step ([8][d][G padded to fours]).
// A thread owns four neighbouring slots, a warp two of the step's queries: per channel one 16-byte load of four key
// elements and two of four heads' query elements feed 32 FMAs.  Per (slot, query) the heads are summed in ascending order
// and the dot products in ascending channel order; the fixed-point window sums of the four warps are integers and are
// added at the end.
constexpr int WR_SLOTS = 128, WR_KPAD = WR_SLOTS + 4, WR_Q = 2, WR_WARPS = 4, WR_STEP = WR_Q * WR_WARPS;
template <typename T>
__global__ void __launch_bounds__(WR_WARPS * 32)
window_ring_grouped_kernel(int G, int kv_heads, int T_len, int d, int w, int B, int cap, float scale, const T* __restrict__ q,
                           int64_t qsb, int64_t qsh, int64_t q_head, int64_t st, const float* __restrict__ lse, int64_t lse_sb,
                           int64_t lse_sh, vatp_cache c) {
  extern __shared__ __align__(16) float wr_smem[];
  const int GP = (G + 3) & ~3;
  float* k_s = wr_smem;                          // [d][WR_KPAD]
  float* q_s = wr_smem + (size_t)d * WR_KPAD;    // [WR_STEP][d][GP]  (16-byte aligned: WR_KPAD is a multiple of four)
  const int u = blockIdx.y, tid = threadIdx.x, lane = tid & 31, wq = tid >> 5;
  const int slot0 = blockIdx.x * WR_SLOTS;
  const int sl4 = lane * 4;                      // this thread's slots: slot0 + sl4 .. + 3
  const int len = min(T_len, B);
  const int b = u / kv_heads, h = u - b * kv_heads;
  const T* qu = q + (int64_t)b * qsb + (int64_t)h * qsh;
  const float* lu = lse + (int64_t)b * lse_sb + (int64_t)h * lse_sh;
  const T* kbase = static_cast<const T*>(c.k_cache) + (int64_t)u * cap * d;
  int ps[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) ps[k] = slot0 + sl4 + k < len ? c.pos[(int64_t)u * cap + slot0 + sl4 + k] : -1;
  const float invG = 1.f / (float)G;
  for (int idx = tid; idx < WR_SLOTS * d; idx += WR_WARPS * 32) {       // consecutive threads: consecutive elements of a row
    const int sl = idx / d, i = idx - sl * d;
    k_s[i * WR_KPAD + sl] = slot0 + sl < cap ? to_f32(kbase[(int64_t)(slot0 + sl) * d + i]) : 0.f;
  }
  for (int idx = tid; idx < WR_STEP * d * GP; idx += WR_WARPS * 32) q_s[idx] = 0.f;      // the padding heads stay zero
  long long fx[4] = {0, 0, 0, 0};
  for (int r0 = 0; r0 < w; r0 += WR_STEP) {
    __syncthreads();
    for (int idx = tid; idx < WR_STEP * G * d; idx += WR_WARPS * 32) {
      const int jj = idx / (G * d), rem = idx - jj * (G * d);
      const int g = rem / d, i = rem - g * d;
      const int j = T_len - w + r0 + jj;
      q_s[(jj * d + i) * GP + g] = (r0 + jj < w && j >= 0) ? to_f32(qu[(int64_t)g * q_head + (int64_t)j * st + i]) : 0.f;
    }
    __syncthreads();
    const int rq = r0 + wq * WR_Q;               // this warp's window rows: rq, rq + 1
    float p[WR_Q][4];
    bool live[WR_Q][4], any = false;
#pragma unroll
    for (int jj = 0; jj < WR_Q; ++jj) {
      const int j = T_len - w + rq + jj;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        p[jj][k] = 0.f;
        // causal: the token precedes the query
        live[jj][k] = slot0 + sl4 + k < cap && rq + jj < w && j >= 0 && ps[k] >= 0 && ps[k] <= j;
        any = any || live[jj][k];
      }
    }
    if (any) {
      for (int g0 = 0; g0 < G; g0 += 4) {
        float a[WR_Q][4][4];                     // [query][head][slot]
#pragma unroll
        for (int jj = 0; jj < WR_Q; ++jj)
#pragma unroll
          for (int hh = 0; hh < 4; ++hh) a[jj][hh][0] = a[jj][hh][1] = a[jj][hh][2] = a[jj][hh][3] = 0.f;
        const float* qw = q_s + (size_t)(wq * WR_Q) * d * GP + g0;
#pragma unroll 2
        for (int i = 0; i < d; ++i) {
          const float4 kv = *reinterpret_cast<const float4*>(&k_s[i * WR_KPAD + sl4]);
#pragma unroll
          for (int jj = 0; jj < WR_Q; ++jj) {
            const float4 qv = *reinterpret_cast<const float4*>(&qw[((size_t)jj * d + i) * GP]);
            const float qh[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
            for (int hh = 0; hh < 4; ++hh) {
              a[jj][hh][0] = fmaf(qh[hh], kv.x, a[jj][hh][0]);
              a[jj][hh][1] = fmaf(qh[hh], kv.y, a[jj][hh][1]);
              a[jj][hh][2] = fmaf(qh[hh], kv.z, a[jj][hh][2]);
              a[jj][hh][3] = fmaf(qh[hh], kv.w, a[jj][hh][3]);
            }
          }
        }
#pragma unroll
        for (int jj = 0; jj < WR_Q; ++jj) {
          const int j = T_len - w + rq + jj;
#pragma unroll
          for (int hh = 0; hh < 4; ++hh) {
            if (g0 + hh < G && rq + jj < w && j >= 0) {
              const float l = __ldg(lu + (int64_t)(g0 + hh) * T_len + j);
#pragma unroll
              for (int k = 0; k < 4; ++k)
                if (live[jj][k]) p[jj][k] += __expf(a[jj][hh][k] * scale - l);
            }
          }
        }
      }
    }
#pragma unroll
    for (int jj = 0; jj < WR_Q; ++jj) {
      const int j = T_len - w + rq + jj;
      if (rq + jj < w) {
        const int rr = ((j % w) + w) % w;
        float* row = c.ring + ((int64_t)u * w + rr) * cap + slot0 + sl4;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (slot0 + sl4 + k < cap) {
            const float pj = live[jj][k] ? p[jj][k] * invG : 0.f;
            row[k] = pj;
            fx[k] += prob_to_fixed(pj);
          }
        }
      }
    }
  }
  __syncthreads();                               // every warp is past its last read of q_s
  long long* fx_s = reinterpret_cast<long long*>(q_s);      // [WR_WARPS][WR_SLOTS]
#pragma unroll
  for (int k = 0; k < 4; ++k) fx_s[wq * WR_SLOTS + sl4 + k] = fx[k];
  __syncthreads();
  const int slot = slot0 + tid;
  if (slot < cap) {
    long long tot = 0;
#pragma unroll
    for (int ww = 0; ww < WR_WARPS; ++ww) tot += fx_s[ww * WR_SLOTS + tid];
    c.acc_fixed[(int64_t)u * cap + slot] = tot;
    c.acc[(int64_t)u * cap + slot] = fixed_to_prob(tot);
  }
}

}  // namespace

// lse: [batch, heads, T] contiguous (every query head's normalisers); s describes the KV units (see make_shape)
cudaError_t launch_window_ring_grouped(const Shape& s, int G, int dtype, int B, const void* q, const float* lse, const vatp_cache& c,
                                       cudaStream_t st) {
  const int cap = cache_capacity(B);
  size_t q_bytes = (size_t)WR_STEP * s.d * ((G + 3) & ~3) * sizeof(float);
  if (q_bytes < (size_t)WR_WARPS * WR_SLOTS * sizeof(long long)) q_bytes = (size_t)WR_WARPS * WR_SLOTS * sizeof(long long);   // the warps' window sums land there at the end
  const size_t smem = (size_t)s.d * WR_KPAD * sizeof(float) + q_bytes;
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
