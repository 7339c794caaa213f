// KV compaction: gather the surviving K and V rows of every unit into the budgeted cache with
// 16-byte loads and stores (bit-exact copies), and initialise the per-slot decode state.
#include "vatp_internal.cuh"

namespace vatp {
namespace {

constexpr int CP_THREADS = 256;
constexpr int CP_ROWS = CP_THREADS / 16;   // rows a CTA copies per step (sixteen lanes per row)
constexpr int CP_ITERS = 4;                // rows of K and of V a thread has in flight before it stores

// One resident wave of CTAs (four per SM).  The destination slots of ALL units form one range of
// units * cap rows, split evenly over the CTAs (to within one row), so that every SM moves the same number
// of bytes whatever the number of units or the budget.  Sixteen lanes copy one row (K and V) in 16-byte pieces;
// a row index costs one 32-bit division per thread and batch of rows.
__global__ void __launch_bounds__(CP_THREADS, 4)
compact_kernel(Shape sh, int elem_bytes, int B, int cap, const char* __restrict__ k, const char* __restrict__ v,
               const float* __restrict__ attn_acc, const float* __restrict__ vnorm, const int32_t* __restrict__ kept,
               vatp_cache c) {
  // launched as a programmatic dependent of the selection: nothing is read before that has completed
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int len = min(sh.T, B);
  const int row_bytes = sh.d * elem_bytes;
  const int hw = threadIdx.x >> 4, l16 = threadIdx.x & 15;
  const int64_t tok_bytes = sh.st * elem_bytes;
  const int64_t total = (int64_t)sh.units * cap;
  const int64_t r_begin = total * blockIdx.x / gridDim.x, r_end = total * (blockIdx.x + 1) / gridDim.x;

  for (int64_t r0 = r_begin + hw; r0 < r_end; r0 += CP_ROWS * CP_ITERS) {
    int src[CP_ITERS], unit[CP_ITERS], slot[CP_ITERS];
#pragma unroll
    for (int i = 0; i < CP_ITERS; ++i) {
      const int64_t r = r0 + i * CP_ROWS;
      unit[i] = -1;
      src[i] = -1;
      slot[i] = 0;
      if (r < r_end) {
        unit[i] = (int)((uint32_t)r / (uint32_t)cap);        // units * cap < 2^32 is checked on the host
        slot[i] = (int)((uint32_t)r - (uint32_t)unit[i] * (uint32_t)cap);
        if (slot[i] < len) src[i] = __ldg(kept + (int64_t)unit[i] * B + slot[i]);
      }
    }
    for (int c0 = l16 * 16; c0 < row_bytes; c0 += 256) {
      uint4 kv[CP_ITERS], vv[CP_ITERS];
#pragma unroll
      for (int i = 0; i < CP_ITERS; ++i) {
        if (src[i] < 0) continue;
        const int64_t o = unit_offset(sh, unit[i]) * elem_bytes + (int64_t)src[i] * tok_bytes + c0;
        kv[i] = __ldg(reinterpret_cast<const uint4*>(k + o));
        vv[i] = __ldg(reinterpret_cast<const uint4*>(v + o));
      }
#pragma unroll
      for (int i = 0; i < CP_ITERS; ++i) {
        if (src[i] < 0) continue;
        const int64_t o = ((int64_t)unit[i] * cap + slot[i]) * row_bytes + c0;
        *reinterpret_cast<uint4*>((char*)c.k_cache + o) = kv[i];
        *reinterpret_cast<uint4*>((char*)c.v_cache + o) = vv[i];
      }
    }
    // per-slot decode state, and the unit's scalars with its first slot
    if (l16 == 0) {
#pragma unroll
      for (int i = 0; i < CP_ITERS; ++i) {
        if (unit[i] < 0) continue;
        const int u = unit[i];
        const int64_t o = (int64_t)u * cap + slot[i];
        c.pos[o] = src[i];
        c.acc[o] = src[i] >= 0 ? __ldg(attn_acc + (int64_t)u * sh.T + src[i]) : 0.f;
        c.vnorm[o] = src[i] >= 0 ? __ldg(vnorm + (int64_t)u * sh.T + src[i]) : 0.f;
        if (slot[i] == 0) {
          c.len[u] = len;
          c.free_slot[u] = len;
          c.next_pos[u] = sh.T;
          c.last_slot[u] = -1;
        }
      }
    }
  }
}

// Windowed indicator state: ring[u][(T - w + r) mod w][slot] = win_rows[u][r][kept[slot]] and the
// exact fixed-point window sum of every slot (Eq. 3).
__global__ void ring_kernel(int units, int T, int w, int B, int cap, const float* __restrict__ win_rows,
                            const int32_t* __restrict__ kept, vatp_cache c) {
  const int u = blockIdx.y;
  const int slot = blockIdx.x * blockDim.x + threadIdx.x;
  if (slot >= cap) return;
  const int len = min(T, B);
  const int src = slot < len ? kept[(int64_t)u * B + slot] : -1;
  long long fx = 0;
  for (int r = 0; r < w; ++r) {
    const int j = T - w + r;                 // query position of this window row (may be < 0)
    const int rr = ((j % w) + w) % w;
    float p = 0.f;
    if (src >= 0 && j >= 0) p = win_rows[((int64_t)u * w + r) * T + src];
    c.ring[((int64_t)u * w + rr) * cap + slot] = p;
    fx += prob_to_fixed(p);
  }
  c.acc_fixed[(int64_t)u * cap + slot] = fx;
  c.acc[(int64_t)u * cap + slot] = fixed_to_prob(fx);
}

}  // namespace

cudaError_t launch_compact(const Shape& s, int dtype, int B, const void* k, const void* v, const float* attn_acc,
                           const float* vnorm, const float* win_rows, const int32_t* kept, const vatp_cache& c,
                           cudaStream_t st) {
  const int eb = dtype == VATP_F32 ? 4 : 2;
  const int cap = cache_capacity(B);
  const int sms = device_sm_count();
  if ((int64_t)s.units * cap >= ((int64_t)1 << 32)) return cudaErrorInvalidValue;
  const int64_t steps = ((int64_t)s.units * cap + CP_ROWS - 1) / CP_ROWS;
  const int64_t wave = 4 * (int64_t)sms;        // four CTAs fit on an SM
  const dim3 grid((unsigned)(steps < wave ? steps : wave));
  DependentLaunch dl(grid, dim3(CP_THREADS), 0, st);
  cudaError_t e = cudaLaunchKernelEx(&dl.cfg, compact_kernel, s, eb, B, cap, (const char*)k, (const char*)v, attn_acc, vnorm,
                                     kept, c);
  if (e != cudaSuccess) return e;
  if (s.window > 0) {
    ring_kernel<<<dim3((cap + 127) / 128, s.units), 128, 0, st>>>(s.units, s.T, s.window, B, cap, win_rows, kept, c);
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace vatp
