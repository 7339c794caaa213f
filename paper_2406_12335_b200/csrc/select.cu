// Budgeted selection: per unit, the top (B - F - R) scores of the middle range [F, T - R) by a
// block-wide radix select on the fp32 bit pattern, ties resolved towards the lower index, and
// the kept indices written in ascending order (first F, selected middle, last R).
// One CTA per unit; the unit's scores are staged in shared memory once when they fit and read
// from global memory (L2-resident) otherwise; for long prompts and few units a cluster of four or two CTAs shares a
// unit (select_cluster_kernel below).  Pure integer work after the key transform.
// Every warp counts into a histogram of its own and the 32 histograms are summed per bin.  The scores
// of a head share a few exponents, so in the first passes nearly all keys of a warp fall into one bin:
// the lanes that agree with the warp's first candidate are counted by one addition (a ballot), the
// others by shared-memory atomics, which rarely collide once the digits spread.  (Grouping all equal
// digits with match.any cost more than everything else in the kernel: it takes time in proportion to
// the number of distinct values in the warp.)
#include <cooperative_groups.h>

#include "vatp_internal.cuh"

namespace cg = cooperative_groups;

namespace vatp {
namespace {

constexpr int SEL_THREADS = 1024;
constexpr int SEL_WARPS = SEL_THREADS / 32;

// order-preserving map float -> uint32 (larger float = larger key), valid for any sign
__device__ __forceinline__ uint32_t order_key(float x) {
  uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

template <bool STAGED>
__global__ void __launch_bounds__(SEL_THREADS) select_kernel(int T, int B, int F, int R, const float* __restrict__ score,
                                                             int32_t* __restrict__ kept, int32_t* dev_status) {
  extern __shared__ __align__(16) uint32_t keys_s[];  // STAGED: keys of the middle range (from index `pad` on)
  __shared__ uint32_t hist[256];
  __shared__ uint32_t hist_w[SEL_WARPS][256];      // per-warp counts of the current pass
  __shared__ uint32_t sh_prefix, sh_need;
  __shared__ uint32_t warp_keep[SEL_WARPS], warp_eq[SEL_WARPS];

  // Launched as a programmatic dependent: the next launch (the compaction) may set up now, and the
  // scores are read only once the launch that produced them has completed.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int u = blockIdx.x;
  const float* sc = score + (int64_t)u * T;
  int32_t* out = kept + (int64_t)u * B;
  const int tid = threadIdx.x;

  if (T <= B) {  // everything survives
    for (int i = tid; i < B; i += SEL_THREADS) out[i] = i < T ? i : -1;
    return;
  }
  const int n = T - R - F;   // middle range length (> 0 here because T > B >= F + R)
  const int ksel = B - F - R;  // how many of the middle range survive
  for (int i = tid; i < F; i += SEL_THREADS) out[i] = i;
  for (int i = tid; i < R; i += SEL_THREADS) out[B - R + i] = T - R + i;
  if (ksel == 0) return;

  // Staging: key i sits at keys_s[pad + i], pad chosen so that 16-byte loads from global memory pair with
  // 16-byte stores to shared memory.  Several loads per thread are in flight at once: one CTA has to pull the
  // whole unit through one SM, and with one 4-byte load per thread in flight that took longer than all the
  // rest of the kernel.
  int pad = 0;
  if (STAGED) {
    const float* mid = sc + F;
    const int a0 = min((int)(((16u - (uint32_t)(reinterpret_cast<uintptr_t>(mid) & 15u)) & 15u) >> 2), n);   // scalars before alignment
    pad = (4 - a0) & 3;
    const int nvec = (n - a0) >> 2;
    const float4* src4 = reinterpret_cast<const float4*>(mid + a0);
    uint4* dst4 = reinterpret_cast<uint4*>(keys_s + pad + a0);
    for (int v0 = 0; v0 < nvec; v0 += 4 * SEL_THREADS) {
      float4 x[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int v = v0 + j * SEL_THREADS + tid;
        if (v < nvec) x[j] = __ldg(src4 + v);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int v = v0 + j * SEL_THREADS + tid;
        if (v < nvec && VATP_INB(pad + a0 + 4 * v + 3, n + 4, dev_status)) dst4[v] = make_uint4(order_key(x[j].x), order_key(x[j].y), order_key(x[j].z), order_key(x[j].w));
      }
    }
    if (tid < a0) keys_s[pad + tid] = order_key(mid[tid]);
    const int tail0 = a0 + 4 * nvec;
    if (tid < n - tail0) keys_s[pad + tail0 + tid] = order_key(mid[tail0 + tid]);
    __syncthreads();
  }
  auto key_at = [&](int i) -> uint32_t { return STAGED ? keys_s[pad + i] : order_key(sc[F + i]); };

  // radix select, most significant byte first: find the key value tau of rank ksel (descending).
  // Lanes that share the digit of the warp's first candidate are counted together; the rest add one each.
  uint32_t prefix = 0, mask = 0, need = (uint32_t)ksel;
  const int lane = tid & 31, wid = tid >> 5;
  for (int shift = 24; shift >= 0; shift -= 8) {
#pragma unroll
    for (int i = lane; i < 256; i += 32) hist_w[wid][i] = 0;
    __syncwarp();
    for (int base = 0; base < n; base += SEL_THREADS) {
      const int i = base + tid;
      uint32_t digit = 256u;                       // lanes without a candidate share a dummy digit
      if (i < n) {
        const uint32_t key = key_at(i);
        if ((key & mask) == prefix) digit = (key >> shift) & 255u;
      }
      const uint32_t cand = __ballot_sync(0xffffffffu, digit < 256u);
      if (cand) {
        const int first = __ffs(cand) - 1;
        const uint32_t d0 = __shfl_sync(0xffffffffu, digit, first);
        const uint32_t same = __ballot_sync(0xffffffffu, digit == d0);
        if (lane == first) atomicAdd(&hist_w[wid][d0], (uint32_t)__popc(same));
        else if (digit < 256u && digit != d0) atomicAdd(&hist_w[wid][digit], 1u);
      }
    }
    __syncthreads();
    if (tid < 256) {
      uint32_t tot = 0;
#pragma unroll 8
      for (int w = 0; w < SEL_WARPS; ++w) tot += hist_w[w][tid];
      hist[tid] = tot;
    }
    __syncthreads();
    if (tid < 32) {
      // walk the 256 bins from the top: 8 bins per lane, suffix sums by shuffles
      uint32_t c[8], tot = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { c[j] = hist[255 - (tid * 8 + j)]; tot += c[j]; }
      uint32_t incl = tot;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, incl, off);
        if (tid >= off) incl += y;
      }
      uint32_t before = incl - tot;  // keys in strictly higher bins than this lane's first bin
      if (before < need && need <= incl) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (need <= before + c[j]) {
            sh_prefix = prefix | ((uint32_t)(255 - (tid * 8 + j)) << shift);
            sh_need = need - before;
            break;
          }
          before += c[j];
        }
      }
    }
    __syncthreads();
    prefix = sh_prefix;
    need = sh_need;
    mask |= 255u << shift;
  }
  const uint32_t tau = prefix;     // the ksel-th largest key; `need` of the keys equal to tau survive
  const uint32_t need_eq = need;

  // Ordered compaction: keep key > tau, and the first need_eq (lowest index) keys equal to tau.
  // Warp w owns the contiguous range [w * per_w, (w + 1) * per_w) and walks it 32 consecutive keys at a time
  // (consecutive shared-memory words: no bank conflicts; one key per lane and a ballot give the order inside a
  // step).  First the warps count their kept and tied keys, one scan over the 32 warp totals gives every warp its
  // output offset and the rank of its first tie, then the warps write.
  const int per_w = ((n + SEL_WARPS - 1) / SEL_WARPS + 31) & ~31;
  const int lo = min(wid * per_w, n), hi_i = min(lo + per_w, n);
  const uint32_t lt_mask = (1u << lane) - 1u;
  uint32_t n_gt = 0, n_eq = 0;                      // warp-uniform
  for (int i0 = lo; i0 < hi_i; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < hi_i ? key_at(i) : 0u;
    n_gt += __popc(__ballot_sync(0xffffffffu, i < hi_i && key > tau));
    n_eq += __popc(__ballot_sync(0xffffffffu, i < hi_i && key == tau));
  }
  if (lane == 0) { warp_keep[wid] = n_gt; warp_eq[wid] = n_eq; }
  __syncthreads();
  // exclusive prefix over the warps, computed by every warp for itself
  uint32_t a = lane < wid ? warp_keep[lane] : 0u, b = lane < wid ? warp_eq[lane] : 0u;
#pragma unroll
  for (int off = 16; off; off >>= 1) {
    a += __shfl_xor_sync(0xffffffffu, a, off);
    b += __shfl_xor_sync(0xffffffffu, b, off);
  }
  uint32_t eq_rank = b;                             // ties before this warp's range
  uint32_t o = a + min(eq_rank, need_eq);           // output offset of this warp's first kept key
  for (int i0 = lo; i0 < hi_i; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < hi_i ? key_at(i) : 0u;
    const bool is_eq = i < hi_i && key == tau;
    const uint32_t eq_b = __ballot_sync(0xffffffffu, is_eq);
    const bool keep = i < hi_i && (key > tau || (is_eq && eq_rank + __popc(eq_b & lt_mask) < need_eq));
    const uint32_t keep_b = __ballot_sync(0xffffffffu, keep);
    if (keep && VATP_INB(F + o + __popc(keep_b & lt_mask), B - R, dev_status)) out[F + o + __popc(keep_b & lt_mask)] = F + i;
    o += __popc(keep_b);
    eq_rank += __popc(eq_b);
  }
}


// ---- the same selection with a unit's middle range split over a cluster of CTAs -------------------------------
// For long prompts and few units one CTA per unit leaves most of the machine idle and counts 32 keys per thread and
// pass.  Here SPLIT CTAs take a contiguous quarter (or half) of the range each: a CTA counts its own keys, pushes its
// 256 bin totals into every partner's shared memory, and after one cluster barrier per pass all CTAs walk the same summed
// histogram to the same digit.  For the ordered write the CTAs exchange how many larger and how many equal keys they hold.
constexpr int SEL_MAXSPLIT = 4;
struct SelExchange {
  uint32_t hist[2][SEL_MAXSPLIT][256];     // per pass parity and rank: that CTA's bin totals
  uint32_t n_gt[SEL_MAXSPLIT], n_eq[SEL_MAXSPLIT];
};
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

__global__ void __launch_bounds__(SEL_THREADS) select_cluster_kernel(int T, int B, int F, int R, int split, int per,
                                                                     const float* __restrict__ score, int32_t* __restrict__ kept,
                                                                     int32_t* dev_status) {
  extern __shared__ __align__(16) uint32_t keys_s[];  // keys of this CTA's part of the middle range
  __shared__ uint32_t hist[256];
  __shared__ uint32_t hist_w[SEL_WARPS][256];
  __shared__ uint32_t sh_prefix, sh_need;
  __shared__ uint32_t warp_keep[SEL_WARPS], warp_eq[SEL_WARPS];
  __shared__ SelExchange xch;

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int u = blockIdx.x / split;
  const float* sc = score + (int64_t)u * T;
  int32_t* out = kept + (int64_t)u * B;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  // (the host uses this kernel only when T > B and B - F - R > 0: every CTA passes every cluster barrier below)
  const int n = T - R - F;     // middle range length
  const int ksel = B - F - R;  // how many of the middle range survive
  // Remote shared memory may only be touched once its CTA runs: everyone arrives here and waits before the first remote store.
  cluster_arrive_release();
  if (rank == 0) {
    for (int i = tid; i < F; i += SEL_THREADS) out[i] = i;
    for (int i = tid; i < R; i += SEL_THREADS) out[B - R + i] = T - R + i;
  }
  const int lo_c = min(rank * per, n), hi_c = min(lo_c + per, n), n_c = hi_c - lo_c;    // this CTA's keys [lo_c, hi_c)
  for (int i = tid; i < n_c; i += SEL_THREADS) keys_s[i] = order_key(__ldg(sc + F + lo_c + i));
  __syncthreads();
  cluster_wait_acquire();

  uint32_t prefix = 0, mask = 0, need = (uint32_t)ksel;
  int pass = 0;
  for (int shift = 24; shift >= 0; shift -= 8, ++pass) {
#pragma unroll
    for (int i = lane; i < 256; i += 32) hist_w[wid][i] = 0;
    __syncwarp();
    for (int base = 0; base < n_c; base += SEL_THREADS) {
      const int i = base + tid;
      uint32_t digit = 256u;                       // lanes without a candidate share a dummy digit
      if (i < n_c) {
        const uint32_t key = keys_s[i];
        if ((key & mask) == prefix) digit = (key >> shift) & 255u;
      }
      const uint32_t cand = __ballot_sync(0xffffffffu, digit < 256u);
      if (cand) {
        const int first = __ffs(cand) - 1;
        const uint32_t d0 = __shfl_sync(0xffffffffu, digit, first);
        const uint32_t same = __ballot_sync(0xffffffffu, digit == d0);
        if (lane == first) atomicAdd(&hist_w[wid][d0], (uint32_t)__popc(same));
        else if (digit < 256u && digit != d0) atomicAdd(&hist_w[wid][digit], 1u);
      }
    }
    __syncthreads();
    if (tid < 256) {
      uint32_t tot = 0;
#pragma unroll 8
      for (int w = 0; w < SEL_WARPS; ++w) tot += hist_w[w][tid];
      for (int r = 0; r < split; ++r) cluster.map_shared_rank(&xch, r)->hist[pass & 1][rank][tid] = tot;
    }
    cluster_arrive_release();
    cluster_wait_acquire();
    if (tid < 256) {
      uint32_t tot = 0;
      for (int r = 0; r < split; ++r) tot += xch.hist[pass & 1][r][tid];
      hist[tid] = tot;
    }
    __syncthreads();
    if (tid < 32) {
      // walk the 256 bins from the top: 8 bins per lane, suffix sums by shuffles
      uint32_t c[8], tot = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { c[j] = hist[255 - (tid * 8 + j)]; tot += c[j]; }
      uint32_t incl = tot;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, incl, off);
        if (tid >= off) incl += y;
      }
      uint32_t before = incl - tot;  // keys in strictly higher bins than this lane's first bin
      if (before < need && need <= incl) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (need <= before + c[j]) {
            sh_prefix = prefix | ((uint32_t)(255 - (tid * 8 + j)) << shift);
            sh_need = need - before;
            break;
          }
          before += c[j];
        }
      }
    }
    __syncthreads();
    prefix = sh_prefix;
    need = sh_need;
    mask |= 255u << shift;
  }
  const uint32_t tau = prefix;     // the ksel-th largest key; `need` of the keys equal to tau survive
  const uint32_t need_eq = need;

  // Ordered compaction as in the single-CTA kernel, over this CTA's part; the CTAs before it in the range tell it how
  // many larger and how many equal keys precede its first one.
  const int per_w = ((n_c + SEL_WARPS - 1) / SEL_WARPS + 31) & ~31;
  const int lo = min(wid * per_w, n_c), hi_i = min(lo + per_w, n_c);
  const uint32_t lt_mask = (1u << lane) - 1u;
  uint32_t n_gt = 0, n_eq = 0;                      // warp-uniform
  for (int i0 = lo; i0 < hi_i; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < hi_i ? keys_s[i] : 0u;
    n_gt += __popc(__ballot_sync(0xffffffffu, i < hi_i && key > tau));
    n_eq += __popc(__ballot_sync(0xffffffffu, i < hi_i && key == tau));
  }
  if (lane == 0) { warp_keep[wid] = n_gt; warp_eq[wid] = n_eq; }
  __syncthreads();
  if (tid == 0) {
    uint32_t g = 0, e = 0;
    for (int w = 0; w < SEL_WARPS; ++w) { g += warp_keep[w]; e += warp_eq[w]; }
    for (int r = 0; r < split; ++r) {
      SelExchange* x = cluster.map_shared_rank(&xch, r);
      x->n_gt[rank] = g;
      x->n_eq[rank] = e;
    }
  }
  cluster_arrive_release();
  cluster_wait_acquire();
  uint32_t base_gt = 0, base_eq = 0;
  for (int r = 0; r < rank; ++r) { base_gt += xch.n_gt[r]; base_eq += xch.n_eq[r]; }
  // exclusive prefix over the warps, computed by every warp for itself
  uint32_t a = lane < wid ? warp_keep[lane] : 0u, b = lane < wid ? warp_eq[lane] : 0u;
#pragma unroll
  for (int off = 16; off; off >>= 1) {
    a += __shfl_xor_sync(0xffffffffu, a, off);
    b += __shfl_xor_sync(0xffffffffu, b, off);
  }
  uint32_t eq_rank = base_eq + b;                   // ties before this warp's range
  uint32_t o = base_gt + a + min(eq_rank, need_eq); // output offset of this warp's first kept key
  for (int i0 = lo; i0 < hi_i; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < hi_i ? keys_s[i] : 0u;
    const bool is_eq = i < hi_i && key == tau;
    const uint32_t eq_b = __ballot_sync(0xffffffffu, is_eq);
    const bool keep = i < hi_i && (key > tau || (is_eq && eq_rank + __popc(eq_b & lt_mask) < need_eq));
    const uint32_t keep_b = __ballot_sync(0xffffffffu, keep);
    if (keep && VATP_INB(F + o + __popc(keep_b & lt_mask), B - R, dev_status)) out[F + o + __popc(keep_b & lt_mask)] = F + lo_c + i;
    o += __popc(keep_b);
    eq_rank += __popc(eq_b);
  }
  // nobody's shared memory is touched after the last barrier above: the CTAs may retire independently
}

}  // namespace

cudaError_t launch_select(int units, int T, int B, int F, int R, const float* score, int32_t* kept, int32_t* dev_status,
                          cudaStream_t st) {
  const int n = T > B ? T - R - F : 0;
  // long prompts, few units: the middle range of a unit goes to a cluster of four or two CTAs
  const int sms = device_sm_count();
  const int split = n >= 8192 && B - F - R > 0 ? (units * 4 <= sms ? 4 : (units * 2 <= sms ? 2 : 1)) : 1;
  if (split > 1) {
    const int per = ((n + split - 1) / split + 31) / 32 * 32;
    const size_t cbytes = (size_t)per * sizeof(uint32_t);
    cudaError_t e = cudaFuncSetAttribute(select_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cbytes);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(units * split);
    cfg.blockDim = dim3(SEL_THREADS);
    cfg.dynamicSmemBytes = cbytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = split;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, select_cluster_kernel, T, B, F, R, split, per, score, kept, dev_status);
  }
  const size_t bytes = (size_t)(n + 4) * sizeof(uint32_t);     // up to three words of alignment padding
  if (bytes <= 160 * 1024) {      // beside the 33 KB of histograms
    cudaError_t e = cudaFuncSetAttribute(select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) return e;
    DependentLaunch dl(dim3(units), dim3(SEL_THREADS), bytes, st);
    return cudaLaunchKernelEx(&dl.cfg, select_kernel<true>, T, B, F, R, score, kept, dev_status);
  }
  DependentLaunch dl(dim3(units), dim3(SEL_THREADS), 0, st);
  return cudaLaunchKernelEx(&dl.cfg, select_kernel<false>, T, B, F, R, score, kept, dev_status);
}

}  // namespace vatp
