// Decode step for grouped-query attention: the G query heads of a KV group attend over ONE shared, budgeted
// cache.  The paper leaves this case to future work ("Compatibility with grouped-query attention") and points
// at a group-wise score; here the indicator of a cached token advances by the MEAN of the probabilities the
// group's heads give it (Eq. 2 under that mean; with a history window, Eq. 3: that mean row enters the ring
// and the exact fixed-point window sum moves by it), Eq. 4 multiplies by the norm of the shared value row, and
// the lowest importance is released as in the multi-head step.
//
// (bf16 with head_dim 128 and up to eight heads per group takes the tensor-core step of decode_mma.cu instead.)
// A general kernel (any dtype and head_dim; CTAs of 512 threads, the probabilities of all heads in shared memory), laid
// out so that every K and V row is read ONCE for all heads of the group.  A unit's slots are split over a cluster of
// four or two CTAs while the grid still fits the SMs at once: every CTA forms the maxima, sums and partial outputs of
// its slots, pushes them into its partners' shared memory, and after one cluster barrier knows the heads' normalisers;
// rank 0 writes the outputs, every CTA updates the indicators of its own slots and proposes an eviction candidate, a
// second barrier, rank 0 picks.
//   logits   the 16-byte pieces of a row go to neighbouring threads (a coalesced read), a warp takes 32 / (pieces
//            per row) rows at a time; a thread forms its piece's share of all G heads' dot products (its pieces of
//            the queries in registers), shuffles add the shares up;
//   softmax  per head over the slots (block reductions);
//   output   the same thread-to-row layout over V: a thread accumulates, for every head, the outputs of its
//            piece's channels; shuffles merge a warp's rows, shared memory the sixteen warps;
//   indicator update and arg-min over the slots as in the multi-head step.
// (The first version walked K once per head from one thread per slot and V once per head and channel, serially:
// 1.8 ms per step for 64 units of 2049 slots; this one takes 43 us.)
#include <cooperative_groups.h>

#include "vatp_internal.cuh"

namespace cg = cooperative_groups;

namespace vatp {
namespace {

__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

constexpr int GQ_THREADS = 512;
constexpr int GQ_WARPS = GQ_THREADS / 32;
constexpr int GQ_FLY = 8;              // row steps a thread requests before it uses the first

__device__ __forceinline__ float block_max(float x, float* red) {
#pragma unroll
  for (int o = 16; o; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
  __syncthreads();
  float y = red[0];
  for (int i = 1; i < GQ_WARPS; ++i) y = fmaxf(y, red[i]);
  return y;
}
__device__ __forceinline__ float block_sum(float x, float* red) {
#pragma unroll
  for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
  __syncthreads();
  float y = 0.f;
  for (int i = 0; i < GQ_WARPS; ++i) y += red[i];      // fixed order
  return y;
}

// the 16-byte piece of a row starting at element e: EP = 8 bf16 or 4 fp32 values, as fp32
template <typename T>
struct Piece;
template <>
struct Piece<__nv_bfloat16> {
  static constexpr int EP = 8;
  __device__ static void load(const __nv_bfloat16* row, int e, float (&x)[8]) {
    const uint4 r = *reinterpret_cast<const uint4*>(row + e);
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { x[2 * i] = __uint_as_float(w[i] << 16); x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
  }
};
template <>
struct Piece<float> {
  static constexpr int EP = 4;
  __device__ static void load(const float* row, int e, float (&x)[4]) {
    const float4 r = *reinterpret_cast<const float4*>(row + e);
    x[0] = r.x; x[1] = r.y; x[2] = r.z; x[3] = r.w;
  }
};

// What the CTAs of a unit tell one another when its slots are split over a cluster (of up to GQ_MAXSPLIT CTAs).
constexpr int GQ_MAXSPLIT = 4;
struct GqExchange {
  float m[GQ_MAXSPLIT][16], l[GQ_MAXSPLIT][16];                  // in every CTA: per rank and head, the maximum of its logits and the sum of exp(x - m)
  unsigned long long key[GQ_MAXSPLIT];       // in rank 0: every rank's eviction candidate (~0: none), its slot and position
  int key_slot[GQ_MAXSPLIT], key_pos[GQ_MAXSPLIT];
};

// GT: compile-time bound on the heads per group (G <= GT): the per-head accumulators stay in registers.
// TPR: threads per row = 16-byte pieces per row when known at compile time (8, 16, 32), 0: taken from d at run time.
// split: CTAs per unit (a cluster of 1, 2 or 4): each takes a contiguous range of `seg` slots.
template <typename T, int GT, int TPR>
__global__ void __launch_bounds__(GQ_THREADS)
decode_gqa_kernel(int G, int d, int B, int cap, int F, int R, int w, int norm, float scale, int split, int seg, vatp_cache c,
                  const T* __restrict__ q_new, const T* __restrict__ k_new, const T* __restrict__ v_new, T* __restrict__ out,
                  int32_t* __restrict__ evicted, int32_t* dev_status) {
  extern __shared__ __align__(16) float gq_smem[];   // p[G][seg] (logits, then exp(x - m)) | q[G][d] | part[warps][G][d] | xo[split][G][d]
  __shared__ float red[GQ_WARPS];
  __shared__ unsigned long long key_red[GQ_WARPS];
  __shared__ int slot_red[GQ_WARPS], pos_red[GQ_WARPS];
  __shared__ GqExchange xch;
  __shared__ float m_loc[16], l_loc[16];
  constexpr int EP = Piece<T>::EP;
  float* p_s = gq_smem;
  float* q_s = gq_smem + (size_t)G * seg;
  float* part_s = q_s + (size_t)G * d;
  float* xo_s = part_s + (size_t)GQ_WARPS * G * d;      // rank 0 receives every rank's partial outputs here
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = split > 1 ? (int)cluster.block_rank() : 0;
  const int u = blockIdx.x / split, tid = threadIdx.x;
  const int len = c.len[u], fs = c.free_slot[u], t = c.next_pos[u];
  if (!VATP_INB(len, cap, dev_status) || !VATP_INB(fs, cap, dev_status)) return;     // (the same verdict in every CTA of the unit)
  // Remote shared memory may only be touched once its CTA runs: everyone arrives here, and waits (long since
  // satisfied) just before the first remote store.
  if (split > 1) cluster_arrive_release();
  const int hi = len + 1;
  const int s_lo = rank * seg, s_hi = min(hi, s_lo + seg);     // this CTA's live slots [s_lo, s_hi)
  T* kc = static_cast<T*>(c.k_cache) + (int64_t)u * cap * d;
  T* vc = static_cast<T*>(c.v_cache) + (int64_t)u * cap * d;

  // ---- append the new token (Eq. 4: its norm) - by the CTA that owns its slot - and stage the group's queries
  const bool owner = fs >= s_lo && fs < s_lo + seg;
  float nn = 0.f;
  for (int i = tid; i < d; i += GQ_THREADS) {
    const T x = v_new[(int64_t)u * d + i];
    if (owner) {
      kc[(int64_t)fs * d + i] = k_new[(int64_t)u * d + i];
      vc[(int64_t)fs * d + i] = x;
    }
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
    for (int i = 1; i < GQ_WARPS; ++i) nn = norm_merge(norm, nn, red[i]);
    nn = norm_finish(norm, nn);
  }
  __syncthreads();                              // the appended rows and the queries are visible to the CTA

  // ---- logits of every head over this CTA's live slots: one row read serves all heads.  tpr = d / EP threads share a
  // row (its 16-byte pieces side by side: a coalesced read), a warp takes 32 / tpr rows at a time; every thread
  // forms the partial dot products of its piece with all G heads, the tpr partials are summed by shuffles.
  const int tpr = TPR ? TPR : d / EP;             // a power of two <= 32 (checked on the host)
  const int rows_w = 32 / tpr;                   // rows per warp and step
  const int lane = tid & 31, wid = tid >> 5;
  const int sub = lane / tpr, piece = lane - sub * tpr;
  {
    float qreg[GT][EP];                          // this thread's piece of every head's query
#pragma unroll
    for (int g = 0; g < GT; ++g)
#pragma unroll
      for (int i = 0; i < EP; ++i) qreg[g][i] = g < G ? q_s[g * d + piece * EP + i] : 0.f;
    // GQ_FLY row steps per thread are requested before any is used: a CTA has to pull its share of the unit through
    // one SM, and with one 16-byte load per thread in flight that took ten times longer than the arithmetic
    const int stride = GQ_WARPS * rows_w;
    for (int s0 = s_lo + wid * rows_w; s0 < s_hi; s0 += GQ_FLY * stride) {
      float x[GQ_FLY][EP];
#pragma unroll
      for (int j = 0; j < GQ_FLY; ++j) {
        const int s = s0 + j * stride + sub;
#pragma unroll
        for (int i = 0; i < EP; ++i) x[j][i] = 0.f;
        if (s < s_hi) Piece<T>::load(kc + (int64_t)s * d, piece * EP, x[j]);
      }
#pragma unroll
      for (int j = 0; j < GQ_FLY; ++j) {
        const int s = s0 + j * stride + sub;
        if (s0 + j * stride >= s_hi) break;          // warp-uniform
        float dot[GT];
#pragma unroll
        for (int g = 0; g < GT; ++g) {
          dot[g] = 0.f;
          if (g < G) {
#pragma unroll
            for (int i = 0; i < EP; ++i) dot[g] = fmaf(qreg[g][i], x[j][i], dot[g]);
#pragma unroll
            for (int o = 16; o; o >>= 1)
              if (o < tpr) dot[g] += __shfl_xor_sync(0xffffffffu, dot[g], o);
          }
        }
        if (piece == 0 && s < s_hi) {
#pragma unroll
          for (int g = 0; g < GT; ++g)
            if (g < G) p_s[(size_t)g * seg + (s - s_lo)] = dot[g] * scale;
        }
      }
    }
  }
  __syncthreads();
  // ---- per head: maximum and sum of exp(x - maximum) over this CTA's slots (Eq. 1; normalised after the exchange)
  const int n_loc = max(s_hi - s_lo, 0);
  for (int g = 0; g < G; ++g) {
    float m = -INFINITY;
    for (int s = tid; s < n_loc; s += GQ_THREADS) m = fmaxf(m, p_s[(size_t)g * seg + s]);
    m = block_max(m, red);
    float l = 0.f;
    for (int s = tid; s < n_loc; s += GQ_THREADS) {
      const float e = __expf(p_s[(size_t)g * seg + s] - m);
      p_s[(size_t)g * seg + s] = e;
      l += e;
    }
    l = block_sum(l, red);
    if (tid == 0) { m_loc[g] = m; l_loc[g] = l; }
  }
  __syncthreads();
  // ---- partial outputs of all heads in one walk over this CTA's value rows: the same thread-to-row layout; a thread
  // holds, for every head, the outputs of its piece's EP channels; rows of one warp are merged by shuffles, the
  // sixteen warps through shared memory.
  {
    float acc[GT][EP];
#pragma unroll
    for (int g = 0; g < GT; ++g)
#pragma unroll
      for (int i = 0; i < EP; ++i) acc[g][i] = 0.f;
    const int stride = GQ_WARPS * rows_w;
    for (int s0 = s_lo + wid * rows_w; s0 < s_hi; s0 += GQ_FLY * stride) {      // GQ_FLY rows in flight per thread
      float x[GQ_FLY][EP];
#pragma unroll
      for (int j = 0; j < GQ_FLY; ++j) {
        const int s = s0 + j * stride + sub;
#pragma unroll
        for (int i = 0; i < EP; ++i) x[j][i] = 0.f;
        if (s < s_hi) Piece<T>::load(vc + (int64_t)s * d, piece * EP, x[j]);
      }
#pragma unroll
      for (int j = 0; j < GQ_FLY; ++j) {
        const int s = s0 + j * stride + sub;
#pragma unroll
        for (int g = 0; g < GT; ++g) {
          if (g < G) {
            const float pj = s < s_hi ? p_s[(size_t)g * seg + (s - s_lo)] : 0.f;
#pragma unroll
            for (int i = 0; i < EP; ++i) acc[g][i] = fmaf(pj, x[j][i], acc[g][i]);
          }
        }
      }
    }
#pragma unroll
    for (int g = 0; g < GT; ++g) {
      if (g < G) {
#pragma unroll
        for (int i = 0; i < EP; ++i) {
          float a = acc[g][i];
#pragma unroll
          for (int o = 16; o; o >>= 1)
            if (o >= tpr) a += __shfl_xor_sync(0xffffffffu, a, o);      // the warp's rows
          if (sub == 0) part_s[((size_t)wid * G + g) * d + piece * EP + i] = a;
        }
      }
    }
    __syncthreads();
    // this CTA's partial output (relative to its own maxima) goes to rank 0, its maxima and sums to every CTA
    if (split > 1) cluster_wait_acquire();
    float* xo0 = split > 1 ? cluster.map_shared_rank(xo_s, 0) : xo_s;
    for (int i = tid; i < G * d; i += GQ_THREADS) {
      float a = 0.f;
      for (int pp = 0; pp < GQ_WARPS; ++pp) a += part_s[(size_t)pp * G * d + i];     // fixed order
      xo0[(size_t)rank * G * d + i] = a;
    }
    if (tid < G * split) {
      const int g = tid % G, r = tid / G;
      GqExchange* xr = split > 1 ? cluster.map_shared_rank(&xch, r) : &xch;
      xr->m[rank][g] = m_loc[g];
      xr->l[rank][g] = l_loc[g];
    }
  }
  if (split > 1) { cluster_arrive_release(); cluster_wait_acquire(); } else __syncthreads();
  // ---- every CTA: the heads' normalisers over the whole unit; sc[g] turns this CTA's exp(x - m) into probabilities
  __shared__ float sc_s[16], fr_s[GQ_MAXSPLIT][16], invL_s[16];
  if (tid < G) {
    const int g = tid;
    float m_all = -INFINITY;
    for (int r = 0; r < split; ++r) m_all = fmaxf(m_all, xch.m[r][g]);
    float L = 0.f;
    for (int r = 0; r < split; ++r) {
      const float f = xch.m[r][g] > -INFINITY ? __expf(xch.m[r][g] - m_all) : 0.f;
      fr_s[r][g] = f;
      L += xch.l[r][g] * f;
    }
    invL_s[g] = 1.f / L;
    sc_s[g] = fr_s[rank][g] / L;
  }
  __syncthreads();
  if (rank == 0) {
    for (int i = tid; i < G * d; i += GQ_THREADS) {
      const int g = i / d;
      float a = 0.f;
      for (int r = 0; r < split; ++r) a = fmaf(xo_s[(size_t)r * G * d + i], fr_s[r][g], a);
      a *= invL_s[g];
      if constexpr (sizeof(T) == 2) out[(int64_t)u * G * d + i] = __float2bfloat16(a);
      else out[(int64_t)u * G * d + i] = a;
    }
  }
  // ---- indicator += mean of the heads' probabilities; importance; arg-min among the unprotected slots (own slots)
  const bool evicting = hi > B;
  unsigned long long my_key = ~0ull;
  int my_slot = -1, my_pos = -1;
  const float invG = 1.f / (float)G;
  for (int s = s_lo + tid; s < s_hi; s += GQ_THREADS) {
    float pm = 0.f;
    for (int g = 0; g < G; ++g) pm = fmaf(p_s[(size_t)g * seg + (s - s_lo)], sc_s[g], pm);
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
  if (owner)
    for (int rr = tid; rr < w; rr += GQ_THREADS)
      if (rr != t % w) c.ring[((int64_t)u * w + rr) * cap + fs] = 0.f;
  if (!evicting) {
    if (rank == 0 && tid == 0) {
      c.len[u] = hi; c.free_slot[u] = hi; c.next_pos[u] = t + 1; c.last_slot[u] = fs;
      if (evicted) evicted[u] = -1;
    }
    return;
  }
  // lowest key of the CTA: warps first, then thread 0 over the warps' candidates; the CTAs' candidates meet in rank 0
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
    for (int i = 0; i < GQ_WARPS; ++i)
      if (key_red[i] < best) { best = key_red[i]; bs = slot_red[i]; bp = pos_red[i]; }
    GqExchange* x0 = split > 1 ? cluster.map_shared_rank(&xch, 0) : &xch;
    x0->key[rank] = best; x0->key_slot[rank] = bs; x0->key_pos[rank] = bp;
  }
  if (split > 1) { cluster_arrive_release(); cluster_wait_acquire(); } else __syncthreads();
  if (rank == 0 && tid == 0) {
    unsigned long long best = ~0ull;
    int bs = -1, bp = -1;
    for (int r = 0; r < split; ++r)
      if (xch.key[r] < best) { best = xch.key[r]; bs = xch.key_slot[r]; bp = xch.key_pos[r]; }
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

template <typename T, int GT, int TPR>
cudaError_t launch_gqa_t(int units, int G, int d, int split, int seg, size_t smem, int B, int cap, int F, int R, int window, int norm,
                         float scale, const vatp_cache& c, const void* q, const void* k, const void* v, void* out, int32_t* evicted,
                         int32_t* dev_status, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(decode_gqa_kernel<T, GT, TPR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(units * split);
  cfg.blockDim = dim3(GQ_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = split;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_gqa_kernel<T, GT, TPR>, G, d, B, cap, F, R, window, norm, scale, split, seg, c,
                            static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), static_cast<T*>(out), evicted,
                            dev_status);
}

// the common row lengths get kernels with the piece count known at compile time
template <typename T, int GT>
cudaError_t launch_gqa(int units, int G, int d, int split, int seg, size_t smem, int B, int cap, int F, int R, int window, int norm,
                       float scale, const vatp_cache& c, const void* q, const void* k, const void* v, void* out, int32_t* evicted,
                       int32_t* dev_status, cudaStream_t st) {
  const int tpr = d / Piece<T>::EP;
  if (tpr == 16) return launch_gqa_t<T, GT, 16>(units, G, d, split, seg, smem, B, cap, F, R, window, norm, scale, c, q, k, v, out, evicted, dev_status, st);
  if (tpr == 8) return launch_gqa_t<T, GT, 8>(units, G, d, split, seg, smem, B, cap, F, R, window, norm, scale, c, q, k, v, out, evicted, dev_status, st);
  return launch_gqa_t<T, GT, 0>(units, G, d, split, seg, smem, B, cap, F, R, window, norm, scale, c, q, k, v, out, evicted, dev_status, st);
}

}  // namespace

cudaError_t launch_group_mean(int G, int64_t n, const float* part, const float* vnorm, float* attn_acc, float* score,
                              cudaStream_t st) {
  group_mean_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(G, n, part, vnorm, attn_acc, score);
  return cudaGetLastError();
}

// units: batch * kv_heads.  cudaErrorNotSupported when the probabilities of a unit's heads do not fit in shared memory,
// for more than 16 heads per group, or for a head_dim whose rows are not a power of two (at most 32) of 16-byte pieces.
cudaError_t launch_decode_gqa(int units, int G, int d, int dtype, int B, int F, int R, int window, int norm, float scale,
                              const vatp_cache& c, const void* q, const void* k, const void* v, void* out, int32_t* evicted,
                              int32_t* dev_status, cudaStream_t st) {
  const int cap = cache_capacity(B);
  const int tpr = d / (dtype == VATP_F32 ? 4 : 8);       // threads that share a row: its 16-byte pieces
  if (G > 16 || d % 8 || tpr < 1 || tpr > 32 || (tpr & (tpr - 1))) return cudaErrorNotSupported;
  // a unit's slots are split over a cluster of four or two CTAs while the grid then still fits on the SMs at once
  const int sms = device_sm_count();
  const int split = units * 4 <= sms ? 4 : (units * 2 <= sms ? 2 : 1);
  const int seg = ((cap + split - 1) / split + 7) / 8 * 8;
  const size_t smem = sizeof(float) * ((size_t)G * seg + (size_t)G * d + (size_t)GQ_WARPS * G * d + (size_t)split * G * d);
  if (smem > 200 * 1024) return cudaErrorNotSupported;
  if (dtype == VATP_F32) {
    if (G <= 4) return launch_gqa<float, 4>(units, G, d, split, seg, smem, B, cap, F, R, window, norm, scale, c, q, k, v, out, evicted, dev_status, st);
    if (G <= 8) return launch_gqa<float, 8>(units, G, d, split, seg, smem, B, cap, F, R, window, norm, scale, c, q, k, v, out, evicted, dev_status, st);
    return launch_gqa<float, 16>(units, G, d, split, seg, smem, B, cap, F, R, window, norm, scale, c, q, k, v, out, evicted, dev_status, st);
  }
  if (G <= 4) return launch_gqa<__nv_bfloat16, 4>(units, G, d, split, seg, smem, B, cap, F, R, window, norm, scale, c, q, k, v, out, evicted, dev_status, st);
  if (G <= 8) return launch_gqa<__nv_bfloat16, 8>(units, G, d, split, seg, smem, B, cap, F, R, window, norm, scale, c, q, k, v, out, evicted, dev_status, st);
  return launch_gqa<__nv_bfloat16, 16>(units, G, d, split, seg, smem, B, cap, F, R, window, norm, scale, c, q, k, v, out, evicted, dev_status, st);
}

}  // namespace vatp
