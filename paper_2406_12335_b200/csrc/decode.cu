// Decode step on the budgeted cache: append the new token, attend (Eq. 1), update the indicator
// (Eq. 2, or the windowed Eq. 3), form the value-aware importance (Eq. 4) and release the
// lowest-importance unprotected slot.
//
// HBM-bound: every cached K and V row is read exactly once per step.  A unit is split over a
// thread-block cluster of SPLIT CTAs (a unit alone cannot fill the machine when there are few
// heads).  Inside a CTA every warp runs its own two-stage pipeline of bulk asynchronous copies
// (global -> shared, completion on an mbarrier): all of a CTA's stages are requested up front, so
// the bytes in flight per SM do not depend on instruction-level latency hiding.  Each half-warp
// keeps an online softmax (running max, sum, partial output), so a V chunk is consumed right after
// its K chunk.  The CTAs of a unit then combine (max, sum, partial output, arg-min candidate)
// through distributed shared memory: no global scratch, no second launch.
#include <cooperative_groups.h>

#include "vatp_internal.cuh"

namespace cg = cooperative_groups;

namespace vatp {
namespace {

constexpr int DEC_THREADS = 256;
constexpr int DEC_WARPS = DEC_THREADS / 32;
constexpr int MAX_SPLIT = 8;
constexpr int ROWS = 8;       // rows of K and of V per pipeline stage
constexpr int NSTAGE = 2;     // stages per warp
constexpr float LOG2E = 1.4426950408889634f;

template <typename T> struct Vec16;  // 16 bytes of T unpacked to floats
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void unpack(const uint4& r, float (&x)[8]) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static void unpack(const uint4& r, float (&x)[4]) {
    x[0] = __uint_as_float(r.x); x[1] = __uint_as_float(r.y); x[2] = __uint_as_float(r.z); x[3] = __uint_as_float(r.w);
  }
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait (about one second): false when the copy never signalled.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  while (!mbar_try_wait(bar, parity))
    if (global_ns() - t0 > 1000000000ull) return false;
  return true;
}
// global -> shared bulk copy; dst, src and bytes are multiples of 16
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

struct Exchange {       // what each CTA publishes to its cluster
  float m, l;           // max of the CTA's logits (log2 domain) and sum of exp2(s - m)
};
struct Candidate {      // arg-min candidate of one CTA, pushed into rank 0's shared memory
  float I;
  int pos, slot;
};

// candidate a is a better eviction choice than b: lower importance, or equal and higher position
__device__ __forceinline__ bool evicts_before(float Ia, int pa, float Ib, int pb) {
  return Ia < Ib || (Ia == Ib && pa > pb);
}

template <typename T, int D, bool WINDOWED>
__global__ void __launch_bounds__(DEC_THREADS)
decode_kernel(int split, int chunk, int B, int cap, int F, int R, int w, int norm, float scale_log2, vatp_cache c,
              const T* __restrict__ q_new, const T* __restrict__ k_new, const T* __restrict__ v_new,
              T* __restrict__ out, int32_t* __restrict__ evicted, int32_t* __restrict__ dev_status) {
  constexpr int EPV = Vec16<T>::N;       // elements per 16-byte vector
  constexpr int LPR = D / EPV;           // lanes per row
  constexpr int RPW = 32 / LPR;          // rows a warp handles at once
  constexpr int NSUB = DEC_WARPS * RPW;  // independent online-softmax partials per CTA
  constexpr int ROWB = D * (int)sizeof(T);
  constexpr int STAGE_BYTES = 2 * ROWS * ROWB;

  extern __shared__ __align__(128) unsigned char dyn_raw[];
  // layout: [DEC_WARPS][NSTAGE][K rows | V rows] | logits[chunk] | acc[chunk] | vnorm[chunk] | pos[chunk]
  unsigned char* stage_base = dyn_raw;
  float* logit_s = reinterpret_cast<float*>(dyn_raw + DEC_WARPS * NSTAGE * STAGE_BYTES);
  float* acc_s = logit_s + chunk;
  float* vn_s = acc_s + chunk;
  int* pos_s = reinterpret_cast<int*>(vn_s + chunk);

  __shared__ __align__(8) uint64_t bars[DEC_WARPS * NSTAGE + 1];
  __shared__ float red_o[NSUB][D];
  __shared__ float sub_m[NSUB], sub_l[NSUB];
  __shared__ float o_cta[D];
  __shared__ Exchange ex;
  __shared__ Candidate cands[MAX_SPLIT];   // used in rank 0 only
  __shared__ float redI[DEC_WARPS];
  __shared__ int redP[DEC_WARPS], redS[DEC_WARPS];

  cg::cluster_group cluster = cg::this_cluster();
  const int rank = split > 1 ? (int)cluster.block_rank() : 0;
  const int u = blockIdx.x / split;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

  // this CTA's slot range inside the allocation (loads do not depend on the live length)
  const int s0 = min(rank * chunk, cap);
  const int rows_alloc = min(chunk, cap - s0);
  const int nchunks = (rows_alloc + ROWS - 1) / ROWS;
  const T* kc = (const T*)c.k_cache + ((int64_t)u * cap + s0) * D;
  const T* vc = (const T*)c.v_cache + ((int64_t)u * cap + s0) * D;
  uint64_t* state_bar = &bars[DEC_WARPS * NSTAGE];

  if (tid == 0) {
    for (int i = 0; i < DEC_WARPS * NSTAGE + 1; ++i) mbar_init(&bars[i], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  auto issue = [&](int ch, int stage) {   // one lane: request K and V rows of chunk `ch`
    const int r0 = ch * ROWS;
    const int n = min(ROWS, rows_alloc - r0);
    unsigned char* dst = stage_base + (wid * NSTAGE + stage) * STAGE_BYTES;
    uint64_t* bar = &bars[wid * NSTAGE + stage];
    mbar_expect_tx(bar, 2u * n * ROWB);
    bulk_g2s(dst, kc + (int64_t)r0 * D, n * ROWB, bar);
    bulk_g2s(dst + ROWS * ROWB, vc + (int64_t)r0 * D, n * ROWB, bar);
  };
  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < NSTAGE; ++s)
      if (wid + s * DEC_WARPS < nchunks) issue(wid + s * DEC_WARPS, s);
  }
  if (tid == 32 && rows_alloc > 0) {      // per-slot state of the range
    const int64_t o = (int64_t)u * cap + s0;
    mbar_expect_tx(state_bar, 3u * rows_alloc * 4u);
    bulk_g2s(acc_s, c.acc + o, rows_alloc * 4, state_bar);
    bulk_g2s(vn_s, c.vnorm + o, rows_alloc * 4, state_bar);
    bulk_g2s(pos_s, c.pos + o, rows_alloc * 4, state_bar);
  }

  const int len = c.len[u];
  const int fs = c.free_slot[u];
  const int t = c.next_pos[u];
  // (bounds-checking build: state words out of range are reported; every access below is clamped to the CTA's rows)
  (void)VATP_INB(len, cap, dev_status);
  (void)VATP_INB(fs, cap, dev_status);
  const int hi = len + 1;                // slots [0, hi) are live once the new token is in
  const int cnt = max(min(hi - s0, rows_alloc), 0);

  const int sub = lane / LPR;            // which of the warp's rows this lane works on
  const int col = (lane % LPR) * EPV;    // first channel of this lane's 16 bytes
  const T* qn = q_new + (int64_t)u * D;
  const T* kn = k_new + (int64_t)u * D;
  const T* vn = v_new + (int64_t)u * D;
  const uint4 kn_raw = *reinterpret_cast<const uint4*>(kn + col);
  const uint4 vn_raw = *reinterpret_cast<const uint4*>(vn + col);
  float qx[EPV];
  Vec16<T>::unpack(*reinterpret_cast<const uint4*>(qn + col), qx);
#pragma unroll
  for (int i = 0; i < EPV; ++i) qx[i] *= scale_log2;

  // ---- append: the CTA that owns the free slot stores the new row and its norm (Eq. 4) ----
  const bool owns_new = fs >= s0 && fs < s0 + cnt;
  float new_norm = 0.f;
  {
    float vx[EPV];
    Vec16<T>::unpack(vn_raw, vx);
#pragma unroll
    for (int i = 0; i < EPV; ++i) new_norm = norm_fold(norm, new_norm, vx[i]);
#pragma unroll
    for (int o = LPR / 2; o; o >>= 1) new_norm = norm_merge(norm, new_norm, __shfl_xor_sync(0xffffffffu, new_norm, o));
    new_norm = norm_finish(norm, new_norm);
  }
  if (owns_new && wid == 0 && sub == 0) {
    *reinterpret_cast<uint4*>((T*)c.k_cache + ((int64_t)u * cap + fs) * D + col) = kn_raw;
    *reinterpret_cast<uint4*>((T*)c.v_cache + ((int64_t)u * cap + fs) * D + col) = vn_raw;
    if (lane == 0) {
      c.vnorm[(int64_t)u * cap + fs] = new_norm;
      c.pos[(int64_t)u * cap + fs] = t;
    }
  }

  // ---- stream the chunks: logits, online softmax, partial output ----
  float m_run = -INFINITY, l_run = 0.f;
  float ox[EPV];
#pragma unroll
  for (int i = 0; i < EPV; ++i) ox[i] = 0.f;
  bool ok = true;
  int it = 0;
  for (int ch = wid; ch < nchunks; ch += DEC_WARPS, ++it) {
    const int stage = it % NSTAGE;
    const uint32_t parity = (it / NSTAGE) & 1;
    if (ok && !mbar_wait(&bars[wid * NSTAGE + stage], parity)) ok = false;
    ok = __all_sync(0xffffffffu, ok);
    const unsigned char* ks = stage_base + (wid * NSTAGE + stage) * STAGE_BYTES;
    const unsigned char* vs = ks + ROWS * ROWB;
    const int r0 = ch * ROWS;
    if (ok && r0 < cnt) {
      float s[ROWS / RPW];
      float cmax = -INFINITY;
#pragma unroll
      for (int j = 0; j < ROWS / RPW; ++j) {
        const int rl = j * RPW + sub;        // row inside the chunk
        const int r = r0 + rl;
        uint4 raw = *reinterpret_cast<const uint4*>(ks + rl * ROWB + col * sizeof(T));
        if (s0 + r == fs) raw = kn_raw;
        float kx[EPV];
        Vec16<T>::unpack(raw, kx);
        float a = 0.f;
#pragma unroll
        for (int i = 0; i < EPV; ++i) a = fmaf(qx[i], kx[i], a);
#pragma unroll
        for (int o = LPR / 2; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        s[j] = r < cnt ? a : -INFINITY;
        if (r < cnt && lane % LPR == 0) logit_s[r] = a;
        cmax = fmaxf(cmax, s[j]);
      }
      const float m_new = fmaxf(m_run, cmax);   // -inf only when every row of this half-warp is masked
      if (m_new > -INFINITY) {
        const float resc = exp2f(m_run - m_new);
        l_run *= resc;
#pragma unroll
        for (int i = 0; i < EPV; ++i) ox[i] *= resc;
#pragma unroll
        for (int j = 0; j < ROWS / RPW; ++j) {
          const int rl = j * RPW + sub;
          const int r = r0 + rl;
          const float e = exp2f(s[j] - m_new);  // 0 for masked rows
          uint4 raw = *reinterpret_cast<const uint4*>(vs + rl * ROWB + col * sizeof(T));
          if (s0 + r == fs) raw = vn_raw;
          float vx[EPV];
          Vec16<T>::unpack(raw, vx);
          l_run += e;
          if (r < cnt) {
#pragma unroll
            for (int i = 0; i < EPV; ++i) ox[i] = fmaf(e, vx[i], ox[i]);
          }
        }
        m_run = m_new;
      }
    }
    __syncwarp();
    const int next = ch + NSTAGE * DEC_WARPS;
    if (ok && lane == 0 && next < nchunks) issue(next, stage);
  }
  if (!ok) {
    // a copy never completed: flag it, give what is still in flight one more bounded wait, carry on
    if (lane == 0) {
      if (dev_status) atomicExch(dev_status, (int)VATP_ERR_TIMEOUT);
      for (int s = 0; s < NSTAGE; ++s) mbar_wait(&bars[wid * NSTAGE + s], 0);
    }
  }
#pragma unroll
  for (int i = 0; i < EPV; ++i) red_o[wid * RPW + sub][col + i] = ox[i];
  if (lane % LPR == 0) { sub_m[wid * RPW + sub] = m_run; sub_l[wid * RPW + sub] = l_run; }
  __syncthreads();

  // ---- CTA partial: max, sum and output over the NSUB partials ----
  float m_c = -INFINITY;
#pragma unroll
  for (int i = 0; i < NSUB; ++i) m_c = fmaxf(m_c, sub_m[i]);
  if (tid < D) {
    float a = 0.f;
#pragma unroll
    for (int i = 0; i < NSUB; ++i)
      if (sub_l[i] > 0.f) a += red_o[i][tid] * exp2f(sub_m[i] - m_c);
    o_cta[tid] = a;
  }
  if (tid == 0) {
    float l = 0.f;
    for (int i = 0; i < NSUB; ++i)
      if (sub_l[i] > 0.f) l += sub_l[i] * exp2f(sub_m[i] - m_c);
    ex.m = m_c;
    ex.l = l;
  }

  // ---- combine the CTAs of the unit ----
  if (split > 1) cluster.sync(); else __syncthreads();
  float m_all = -INFINITY, L = 0.f;
  {
    float ms[MAX_SPLIT], ls[MAX_SPLIT];
#pragma unroll
    for (int r = 0; r < MAX_SPLIT; ++r) {
      ms[r] = -INFINITY; ls[r] = 0.f;
      if (r < split) {
        const Exchange* e = split > 1 ? cluster.map_shared_rank(&ex, r) : &ex;
        ms[r] = e->m; ls[r] = e->l;
      }
      m_all = fmaxf(m_all, ms[r]);
    }
#pragma unroll
    for (int r = 0; r < MAX_SPLIT; ++r)
      if (ls[r] > 0.f) L += ls[r] * exp2f(ms[r] - m_all);
    if (rank == 0 && tid < D) {
      float a = 0.f;
#pragma unroll
      for (int r = 0; r < MAX_SPLIT; ++r) {
        if (r < split && ls[r] > 0.f) {
          const float* o = split > 1 ? cluster.map_shared_rank(o_cta, r) : o_cta;
          a += o[tid] * exp2f(ms[r] - m_all);
        }
      }
      out[(int64_t)u * D + tid] = (T)(a / L);
    }
  }
  const float invL = 1.f / L;

  // ---- indicator update (Eq. 2 / Eq. 3), importance (Eq. 4), local arg-min ----
  if (rows_alloc > 0 && !mbar_wait(state_bar, 0) && dev_status) atomicExch(dev_status, (int)VATP_ERR_TIMEOUT);
  const bool evicting = hi > B;
  float bestI = INFINITY; int bestP = -1, bestS = -1;
  for (int r = tid; r < cnt; r += DEC_THREADS) {
    const int slot = s0 + r;
    const int64_t o = (int64_t)u * cap + slot;
    const float p = exp2f(logit_s[r] - m_all) * invL;
    const bool is_new = slot == fs;
    float S;
    if (WINDOWED) {
      float* ring_row = c.ring + ((int64_t)u * w + (t % w)) * cap;
      long long fx;
      if (is_new) {
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
      S = is_new ? p : acc_s[r] + p;
    }
    c.acc[o] = S;
    if (evicting) {
      const int ps = is_new ? t : pos_s[r];
      const float I = S * (is_new ? new_norm : vn_s[r]);
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
      Candidate cd{INFINITY, -1, -1};
      for (int i = 0; i < DEC_WARPS; ++i)
        if (redS[i] >= 0 && (cd.slot < 0 || evicts_before(redI[i], redP[i], cd.I, cd.pos))) {
          cd.I = redI[i]; cd.pos = redP[i]; cd.slot = redS[i];
        }
      Candidate* dst = split > 1 ? cluster.map_shared_rank(&cands[rank], 0) : &cands[rank];
      *dst = cd;                                  // push into rank 0's shared memory
    }
  }
  if (split > 1) cluster.sync(); else __syncthreads();   // candidates delivered; remote reads of o_cta done
  if (rank == 0 && tid == 0) {
    int ev_pos = -1;
    if (evicting) {
      Candidate best{INFINITY, -1, -1};
      for (int r = 0; r < split; ++r)
        if (cands[r].slot >= 0 && (best.slot < 0 || evicts_before(cands[r].I, cands[r].pos, best.I, best.pos)))
          best = cands[r];
      if (best.slot >= 0) {
        c.pos[(int64_t)u * cap + best.slot] = -1;
        c.free_slot[u] = best.slot;
        c.len[u] = hi - 1;
        ev_pos = best.pos;
      } else {               // nothing eligible (cannot happen when F + R <= B): keep the state consistent
        c.len[u] = hi;
        c.free_slot[u] = min(hi, cap - 1);
      }
    } else {
      c.len[u] = hi;
      c.free_slot[u] = hi;
    }
    c.next_pos[u] = t + 1;
    c.last_slot[u] = fs;
    if (evicted) evicted[u] = ev_pos;
  }
}

template <typename T, int D, bool WINDOWED>
cudaError_t launch_t(const Shape& s, int B, int F, int R, const vatp_cache& c, const void* q, const void* k,
                     const void* v, void* out, int32_t* evicted, int32_t* dev_status, cudaStream_t st) {
  const int cap = cache_capacity(B);
  // split a unit over a cluster when there are too few units to fill 148 SMs
  int split = 1;
  while (split < MAX_SPLIT && s.units * split * 2 <= 148 * 2 && cap / (split * 2) >= 64) split *= 2;
  int chunk = (cap + split - 1) / split;
  chunk = (chunk + 7) / 8 * 8;
  const size_t stage_bytes = (size_t)DEC_WARPS * NSTAGE * 2 * ROWS * D * sizeof(T);
  const size_t dyn = stage_bytes + 4 * sizeof(float) * chunk;
  if (dyn > 200 * 1024) return cudaErrorInvalidConfiguration;
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
  return cudaLaunchKernelEx(&cfg, kern, split, chunk, B, cap, F, R, s.window, s.norm, s.scale * LOG2E, c, (const T*)q,
                            (const T*)k, (const T*)v, (T*)out, evicted, dev_status);
}

}  // namespace

cudaError_t launch_decode(const Shape& s, int dtype, int B, int F, int R, const vatp_cache& c, const void* q,
                          const void* k, const void* v, void* out, int32_t* evicted, int32_t* dev_status,
                          cudaStream_t st, bool may_overlap) {
  const bool win = s.window > 0;
  if (dtype == VATP_BF16 && s.d == 128) {
    const cudaError_t e = launch_decode_mma(s, B, F, R, c, q, k, v, out, evicted, dev_status, st, may_overlap);
    if (e != cudaErrorNotSupported) return e;
  }
  decode_history_forget(st);     // the general kernel is an ordinary launch: the record of overlapping launches ends here
#define VATP_DISPATCH(T, D)                                                                         \
  return win ? launch_t<T, D, true>(s, B, F, R, c, q, k, v, out, evicted, dev_status, st)           \
             : launch_t<T, D, false>(s, B, F, R, c, q, k, v, out, evicted, dev_status, st)
  if (dtype == VATP_F32) {
    if (s.d == 64) { VATP_DISPATCH(float, 64); }
    VATP_DISPATCH(float, 128);
  }
  if (s.d == 64) { VATP_DISPATCH(__nv_bfloat16, 64); }
  VATP_DISPATCH(__nv_bfloat16, 128);
#undef VATP_DISPATCH
}

}  // namespace vatp
