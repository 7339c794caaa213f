// Budgeted selection: per unit, the top (B - F - R) scores of the middle range [F, T - R) by a
// block-wide radix select on the fp32 bit pattern, ties resolved towards the lower index, and
// the kept indices written in ascending order (first F, selected middle, last R).
// One CTA per unit; the unit's scores are staged in shared memory once when they fit and read
// from global memory (L2-resident) otherwise.  Pure integer work after the key transform.
#include "vatp_internal.cuh"

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
                                                             int32_t* __restrict__ kept) {
  extern __shared__ uint32_t keys_s[];  // STAGED: keys of the middle range
  __shared__ uint32_t hist[256];
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

  if (STAGED) {
    for (int i = tid; i < n; i += SEL_THREADS) keys_s[i] = order_key(sc[F + i]);
    __syncthreads();
  }
  auto key_at = [&](int i) -> uint32_t { return STAGED ? keys_s[i] : order_key(sc[F + i]); };

  // radix select, most significant byte first: find the key value tau of rank ksel (descending).
  // Scores of one head share a few exponents, so most keys of a pass fall into a handful of bins:
  // lanes with the same digit are counted by one of them (match + one atomic per distinct digit).
  uint32_t prefix = 0, mask = 0, need = (uint32_t)ksel;
  const int lane = tid & 31, wid = tid >> 5;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += SEL_THREADS) hist[i] = 0;
    __syncthreads();
    for (int base = 0; base < n; base += SEL_THREADS) {
      const int i = base + tid;
      uint32_t digit = 256u;                       // lanes without a candidate share a dummy digit
      if (i < n) {
        const uint32_t key = key_at(i);
        if ((key & mask) == prefix) digit = (key >> shift) & 255u;
      }
      const uint32_t peers = __match_any_sync(0xffffffffu, digit);
      if (digit < 256u && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
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

  // ordered compaction: keep key > tau, and the first need_eq (lowest index) keys equal to tau.
  // Thread t owns the contiguous range [t * per, (t + 1) * per); one block-wide exclusive scan of
  // (kept, equal) counts gives every thread its output offset and the rank of its first tie.
  const int per = (n + SEL_THREADS - 1) / SEL_THREADS;
  const int lo = min(tid * per, n), hi_i = min(lo + per, n);
  uint32_t n_gt = 0, n_eq = 0;
  for (int i = lo; i < hi_i; ++i) {
    const uint32_t key = key_at(i);
    n_gt += key > tau;
    n_eq += key == tau;
  }
  // inclusive scan inside the warp, then over the warp totals
  uint32_t s_gt = n_gt, s_eq = n_eq;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t a = __shfl_up_sync(0xffffffffu, s_gt, off), b = __shfl_up_sync(0xffffffffu, s_eq, off);
    if (lane >= off) { s_gt += a; s_eq += b; }
  }
  if (lane == 31) { warp_keep[wid] = s_gt; warp_eq[wid] = s_eq; }
  __syncthreads();
  if (wid == 0) {
    uint32_t a = warp_keep[lane], b = warp_eq[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t x = __shfl_up_sync(0xffffffffu, a, off), y = __shfl_up_sync(0xffffffffu, b, off);
      if (lane >= off) { a += x; b += y; }
    }
    warp_keep[lane] = a;      // inclusive totals up to and including warp `lane`
    warp_eq[lane] = b;
  }
  __syncthreads();
  const uint32_t gt_before = s_gt - n_gt + (wid ? warp_keep[wid - 1] : 0u);
  uint32_t eq_rank = s_eq - n_eq + (wid ? warp_eq[wid - 1] : 0u);
  // ties before index i that survive = min(eq_rank, need_eq)
  uint32_t o = gt_before + min(eq_rank, need_eq);
  for (int i = lo; i < hi_i; ++i) {
    const uint32_t key = key_at(i);
    const bool keep = key > tau || (key == tau && eq_rank < need_eq);
    eq_rank += key == tau;
    if (keep) out[F + o++] = F + i;
  }
}

}  // namespace

cudaError_t launch_select(int units, int T, int B, int F, int R, const float* score, int32_t* kept, cudaStream_t st) {
  const int n = T > B ? T - R - F : 0;
  const size_t bytes = (size_t)n * sizeof(uint32_t);
  if (bytes <= 200 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) return e;
    DependentLaunch dl(dim3(units), dim3(SEL_THREADS), bytes, st);
    return cudaLaunchKernelEx(&dl.cfg, select_kernel<true>, T, B, F, R, score, kept);
  }
  DependentLaunch dl(dim3(units), dim3(SEL_THREADS), 0, st);
  return cudaLaunchKernelEx(&dl.cfg, select_kernel<false>, T, B, F, R, score, kept);
}

}  // namespace vatp
