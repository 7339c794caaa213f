// Decode step on the budgeted cache: append the new token, attend (Eq. 1), update the indicator
// (Eq. 2, or the windowed Eq. 3), form the value-aware importance (Eq. 4) and release the
// lowest-importance unprotected slot.
//
// HBM-bound: every cached K and V row is read exactly once per step with 16-byte loads.  A unit
// is split over a thread-block cluster of SPLIT CTAs (a unit alone cannot fill the machine when
// there are few heads); each CTA handles a contiguous range of slots with a local softmax, and
// the CTAs combine (max, sum, partial output, arg-min candidate) through distributed shared
// memory, so no global scratch and no second launch is needed.
#include <cooperative_groups.h>

#include "vatp_internal.cuh"

namespace cg = cooperative_groups;

namespace vatp {
namespace {

constexpr int DEC_THREADS = 256;
constexpr int DEC_WARPS = DEC_THREADS / 32;
constexpr int MAX_SPLIT = 8;
constexpr float LOG2E = 1.4426950408889634f;

template <typename T> struct Vec16;  // 16 bytes of T unpacked to floats
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const void* p, float (&x)[8]) {
    const uint4 r = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static void store(void* p, const float (&x)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static void load(const void* p, float (&x)[4]) {
    const float4 r = *reinterpret_cast<const float4*>(p);
    x[0] = r.x; x[1] = r.y; x[2] = r.z; x[3] = r.w;
  }
  __device__ static void store(void* p, const float (&x)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  }
};

struct Exchange {       // what each CTA publishes to its cluster
  float m, l;           // local max of the logits (log2 domain) and sum of exp2(s - m)
  float cand_I;         // arg-min candidate: importance, position, slot (-1 = none)
  int cand_pos, cand_slot;
};

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
// candidate a is a better eviction choice than b: lower importance, or equal and higher position
__device__ __forceinline__ bool evicts_before(float Ia, int pa, float Ib, int pb) {
  return Ia < Ib || (Ia == Ib && pa > pb);
}

template <typename T, int D, bool WINDOWED>
__global__ void __launch_bounds__(DEC_THREADS)
decode_kernel(int split, int chunk, int B, int F, int R, int w, float scale_log2, vatp_cache c,
              const T* __restrict__ q_new, const T* __restrict__ k_new, const T* __restrict__ v_new,
              T* __restrict__ out, int32_t* __restrict__ evicted) {
  constexpr int EPV = Vec16<T>::N;       // elements per 16-byte vector
  constexpr int LPR = D / EPV;           // lanes per row
  constexpr int RPW = 32 / LPR;          // rows per warp pass
  extern __shared__ float dyn[];         // [chunk] logits, then exp2 values
  __shared__ float red_o[DEC_WARPS * RPW][D];
  __shared__ float o_cta[D];
  __shared__ float red[DEC_WARPS];
  __shared__ float redI[DEC_WARPS];
  __shared__ int redP[DEC_WARPS], redS[DEC_WARPS];
  __shared__ Exchange ex;
  __shared__ float bc_m, bc_f;

  cg::cluster_group cluster = cg::this_cluster();
  const int rank = split > 1 ? (int)cluster.block_rank() : 0;
  const int u = blockIdx.x / split;
  const int cap = B + 1;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

  const int len = c.len[u];
  const int fs = c.free_slot[u];
  const int t = c.next_pos[u];
  const int hi = len + 1;                // slots [0, hi) are live once the new token is in
  const int s0 = min(rank * chunk, hi), s1 = min(s0 + chunk, hi);
  const int cnt = s1 - s0;

  const T* kc = (const T*)c.k_cache + (int64_t)u * cap * D;
  const T* vc = (const T*)c.v_cache + (int64_t)u * cap * D;
  const T* qn = q_new + (int64_t)u * D;
  const T* kn = k_new + (int64_t)u * D;
  const T* vn = v_new + (int64_t)u * D;
  const int sub = lane / LPR;            // which of the warp's rows this lane works on
  const int col = (lane % LPR) * EPV;    // first channel of this lane's 16 bytes

  // ---- append: the CTA that owns the free slot stores the new row and its l1 norm ----
  const bool owns_new = fs >= s0 && fs < s1;
  if (owns_new && wid == 0) {
    float kx[EPV], vx[EPV];
    if (lane < LPR) {
      Vec16<T>::load(kn + col, kx);
      Vec16<T>::load(vn + col, vx);
      Vec16<T>::store((T*)c.k_cache + ((int64_t)u * cap + fs) * D + col, kx);
      Vec16<T>::store((T*)c.v_cache + ((int64_t)u * cap + fs) * D + col, vx);
    }
    float a = 0.f;
    if (lane < LPR) {
#pragma unroll
      for (int i = 0; i < EPV; ++i) a += fabsf(vx[i]);
    }
    a = warp_sum(a);
    if (lane == 0) {
      c.vnorm[(int64_t)u * cap + fs] = a;
      c.pos[(int64_t)u * cap + fs] = t;
    }
  }

  // ---- logits: s_i = scale * <q, k_i>, kept in the log2 domain ----
  float qx[EPV];
  Vec16<T>::load(qn + col, qx);
#pragma unroll
  for (int i = 0; i < EPV; ++i) qx[i] *= scale_log2;
  float lmax = -INFINITY;
  constexpr int UN = 4;
  for (int r0 = wid * RPW * UN; r0 < cnt; r0 += DEC_WARPS * RPW * UN) {
    float kx[UN][EPV];
#pragma unroll
    for (int j = 0; j < UN; ++j) {
      const int r = r0 + j * RPW + sub;
      if (r < cnt) {
        const int slot = s0 + r;
        const T* src = slot == fs ? kn : kc + (int64_t)slot * D;
        Vec16<T>::load(src + col, kx[j]);
      }
    }
#pragma unroll
    for (int j = 0; j < UN; ++j) {
      const int r = r0 + j * RPW + sub;
      float s = 0.f;
      if (r < cnt) {
#pragma unroll
        for (int i = 0; i < EPV; ++i) s = fmaf(qx[i], kx[j][i], s);
      }
#pragma unroll
      for (int o = LPR / 2; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (r < cnt) {
        if (lane % LPR == 0) dyn[r] = s;
        lmax = fmaxf(lmax, s);
      }
    }
  }
  lmax = warp_max(lmax);
  if (lane == 0) red[wid] = lmax;
  __syncthreads();
  if (tid == 0) {
    float m = -INFINITY;
    for (int i = 0; i < DEC_WARPS; ++i) m = fmaxf(m, red[i]);
    bc_m = m;
  }
  __syncthreads();
  const float m_c = bc_m;                // -inf when this CTA has no slots

  // ---- exp2 and local sum ----
  float lsum = 0.f;
  for (int r = tid; r < cnt; r += DEC_THREADS) {
    const float e = exp2f(dyn[r] - m_c);
    dyn[r] = e;
    lsum += e;
  }
  lsum = warp_sum(lsum);
  __syncthreads();                       // red is reused; dyn[] exp values visible
  if (lane == 0) red[wid] = lsum;

  // ---- partial output: o = sum_i e_i v_i over this CTA's slots ----
  float ox[EPV];
#pragma unroll
  for (int i = 0; i < EPV; ++i) ox[i] = 0.f;
  for (int r0 = wid * RPW * UN; r0 < cnt; r0 += DEC_WARPS * RPW * UN) {
    float vx[UN][EPV];
    float e[UN];
#pragma unroll
    for (int j = 0; j < UN; ++j) {
      const int r = r0 + j * RPW + sub;
      e[j] = 0.f;
      if (r < cnt) {
        const int slot = s0 + r;
        const T* src = slot == fs ? vn : vc + (int64_t)slot * D;
        Vec16<T>::load(src + col, vx[j]);
        e[j] = dyn[r];
      }
    }
#pragma unroll
    for (int j = 0; j < UN; ++j) {
      const int r = r0 + j * RPW + sub;
      if (r < cnt) {
#pragma unroll
        for (int i = 0; i < EPV; ++i) ox[i] = fmaf(e[j], vx[j][i], ox[i]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < EPV; ++i) red_o[wid * RPW + sub][col + i] = ox[i];
  __syncthreads();
  if (tid < D) {
    float a = 0.f;
#pragma unroll
    for (int i = 0; i < DEC_WARPS * RPW; ++i) a += red_o[i][tid];
    o_cta[tid] = a;
  }
  if (tid == 0) {
    float l = 0.f;
    for (int i = 0; i < DEC_WARPS; ++i) l += red[i];
    ex.m = m_c;
    ex.l = l;
  }

  // ---- combine the CTAs of the unit ----
  if (split > 1) cluster.sync(); else __syncthreads();
  if (tid == 0) {
    float m = -INFINITY, L = 0.f;
    float ms[MAX_SPLIT], ls[MAX_SPLIT];
    for (int r = 0; r < split; ++r) {
      const Exchange* e = split > 1 ? cluster.map_shared_rank(&ex, r) : &ex;
      ms[r] = e->m; ls[r] = e->l;
      m = fmaxf(m, ms[r]);
    }
    for (int r = 0; r < split; ++r) if (ls[r] > 0.f) L += ls[r] * exp2f(ms[r] - m);
    bc_m = m;
    bc_f = 1.f / L;
  }
  __syncthreads();
  const float m_all = bc_m, invL = bc_f;
  if (rank == 0 && tid < D) {
    float a = 0.f;
    for (int r = 0; r < split; ++r) {
      const Exchange* e = split > 1 ? cluster.map_shared_rank(&ex, r) : &ex;
      const float* o = split > 1 ? cluster.map_shared_rank(o_cta, r) : o_cta;
      if (e->l > 0.f) a += o[tid] * exp2f(e->m - m_all);
    }
    out[(int64_t)u * D + tid] = (T)(a * invL);
  }

  // ---- indicator update (Eq. 2 / Eq. 3), importance (Eq. 4), local arg-min ----
  const float f = cnt > 0 ? exp2f(m_c - m_all) * invL : 0.f;
  const bool evicting = hi > B;
  float bestI = INFINITY; int bestP = -1, bestS = -1;
  for (int r = tid; r < cnt; r += DEC_THREADS) {
    const int slot = s0 + r;
    const int64_t o = (int64_t)u * cap + slot;
    const float p = dyn[r] * f;
    float S;
    if (WINDOWED) {
      float* ring_row = c.ring + ((int64_t)u * w + (t % w)) * cap;
      long long fx;
      if (slot == fs) {
        // recycled slot: its ring column belongs to the previous occupant
        for (int rr = 0; rr < w; ++rr) c.ring[((int64_t)u * w + rr) * cap + slot] = 0.f;
        fx = prob_to_fixed(p);
      } else {
        fx = c.acc_fixed[o] + prob_to_fixed(p) - prob_to_fixed(ring_row[slot]);
      }
      ring_row[slot] = p;
      c.acc_fixed[o] = fx;
      S = fixed_to_prob(fx);
    } else {
      S = slot == fs ? p : c.acc[o] + p;
    }
    c.acc[o] = S;
    if (evicting) {
      const int ps = slot == fs ? t : c.pos[o];
      const float I = S * c.vnorm[o];
      if (ps >= F && ps <= t - R && evicts_before(I, ps, bestI, bestP)) { bestI = I; bestP = ps; bestS = slot; }
    }
  }
  if (evicting) {
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      const float I2 = __shfl_xor_sync(0xffffffffu, bestI, o);
      const int P2 = __shfl_xor_sync(0xffffffffu, bestP, o);
      const int S2 = __shfl_xor_sync(0xffffffffu, bestS, o);
      if (S2 >= 0 && (bestS < 0 || evicts_before(I2, P2, bestI, bestP))) { bestI = I2; bestP = P2; bestS = S2; }
    }
    if (lane == 0) { redI[wid] = bestI; redP[wid] = bestP; redS[wid] = bestS; }
    __syncthreads();
    if (tid == 0) {
      float bI = INFINITY; int bP = -1, bS = -1;
      for (int i = 0; i < DEC_WARPS; ++i)
        if (redS[i] >= 0 && (bS < 0 || evicts_before(redI[i], redP[i], bI, bP))) { bI = redI[i]; bP = redP[i]; bS = redS[i]; }
      ex.cand_I = bI; ex.cand_pos = bP; ex.cand_slot = bS;
    }
    if (split > 1) cluster.sync(); else __syncthreads();
  }
  if (rank == 0 && tid == 0) {
    int ev_pos = -1;
    if (evicting) {
      float bI = INFINITY; int bP = -1, bS = -1;
      for (int r = 0; r < split; ++r) {
        const Exchange* e = split > 1 ? cluster.map_shared_rank(&ex, r) : &ex;
        if (e->cand_slot >= 0 && (bS < 0 || evicts_before(e->cand_I, e->cand_pos, bI, bP))) {
          bI = e->cand_I; bP = e->cand_pos; bS = e->cand_slot;
        }
      }
      if (bS >= 0) {
        c.pos[(int64_t)u * cap + bS] = -1;
        c.free_slot[u] = bS;
        c.len[u] = hi - 1;
        ev_pos = bP;
      } else {               // nothing eligible (cannot happen when F + R <= B): keep state consistent
        c.len[u] = hi;
        c.free_slot[u] = min(hi, cap - 1);
      }
    } else {
      c.len[u] = hi;
      c.free_slot[u] = hi;
    }
    c.next_pos[u] = t + 1;
    if (evicted) evicted[u] = ev_pos;
  }
  if (split > 1) cluster.sync();   // remote shared memory must outlive the reads above
}

template <typename T, int D, bool WINDOWED>
cudaError_t launch_t(const Shape& s, int B, int F, int R, const vatp_cache& c, const void* q, const void* k,
                     const void* v, void* out, int32_t* evicted, cudaStream_t st) {
  const int cap = B + 1;
  // split a unit over a cluster when there are too few units to fill 148 SMs twice over
  int split = 1;
  while (split < MAX_SPLIT && s.units * split < 2 * 148 && cap / (split * 2) >= 64) split *= 2;
  int chunk = (cap + split - 1) / split;
  chunk = (chunk + 7) / 8 * 8;
  const size_t dyn = sizeof(float) * chunk;
  auto kern = decode_kernel<T, D, WINDOWED>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(s.units * split);
  cfg.blockDim = dim3(DEC_THREADS);
  cfg.dynamicSmemBytes = dyn;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = split;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, split, chunk, B, F, R, s.window, s.scale * LOG2E, c, (const T*)q, (const T*)k,
                            (const T*)v, (T*)out, evicted);
}

}  // namespace

cudaError_t launch_decode(const Shape& s, int dtype, int B, int F, int R, const vatp_cache& c, const void* q,
                          const void* k, const void* v, void* out, int32_t* evicted, cudaStream_t st) {
  const bool win = s.window > 0;
#define VATP_DISPATCH(T, D)                                                             \
  return win ? launch_t<T, D, true>(s, B, F, R, c, q, k, v, out, evicted, st)           \
             : launch_t<T, D, false>(s, B, F, R, c, q, k, v, out, evicted, st)
  if (dtype == VATP_F32) {
    if (s.d == 64) { VATP_DISPATCH(float, 64); }
    VATP_DISPATCH(float, 128);
  }
  if (s.d == 64) { VATP_DISPATCH(__nv_bfloat16, 64); }
  VATP_DISPATCH(__nv_bfloat16, 128);
#undef VATP_DISPATCH
}

}  // namespace vatp
