// KV compaction: gather the surviving K and V rows of every unit into the budgeted cache with
// 16-byte loads and stores (bit-exact copies), and initialise the per-slot decode state.
#include "vatp_internal.cuh"

namespace vatp {
namespace {

constexpr int CP_THREADS = 256;
constexpr int CP_SLOTS = 64;     // destination slots per CTA
constexpr int CP_ITERS = CP_SLOTS / (CP_THREADS / 16);

// grid (units, y), each CTA walking slot groups y, y + gridDim.y, ... so that the whole grid is one
// resident wave.  Sixteen lanes copy one row (K and V) in 16-byte pieces; a thread has CP_ITERS rows of
// K and of V in flight before it stores, and no index needs a division.
__global__ void __launch_bounds__(CP_THREADS, 4)
compact_kernel(Shape sh, int elem_bytes, int B, int cap, const char* __restrict__ k, const char* __restrict__ v,
               const float* __restrict__ attn_acc, const float* __restrict__ vnorm, const int32_t* __restrict__ kept,
               vatp_cache c) {
  // launched as a programmatic dependent of the selection: nothing is read before that has completed
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int u = blockIdx.x;
  const int len = min(sh.T, B);
  const int row_bytes = sh.d * elem_bytes;
  const int hw = threadIdx.x >> 4, l16 = threadIdx.x & 15;
  const int64_t unit_bytes = unit_offset(sh, u) * elem_bytes;
  const int64_t tok_bytes = sh.st * elem_bytes;

  for (int grp = blockIdx.y; grp * CP_SLOTS < cap; grp += gridDim.y) {
  const int slot0 = grp * CP_SLOTS + hw;
  int src[CP_ITERS];
#pragma unroll
  for (int i = 0; i < CP_ITERS; ++i) {
    const int slot = slot0 + i * (CP_THREADS / 16);
    src[i] = slot < len ? __ldg(kept + (int64_t)u * B + slot) : -1;
  }
  for (int c0 = l16 * 16; c0 < row_bytes; c0 += 256) {
    uint4 kv[CP_ITERS], vv[CP_ITERS];
#pragma unroll
    for (int i = 0; i < CP_ITERS; ++i) {
      if (src[i] < 0) continue;
      const int64_t o = unit_bytes + (int64_t)src[i] * tok_bytes + c0;
      kv[i] = __ldg(reinterpret_cast<const uint4*>(k + o));
      vv[i] = __ldg(reinterpret_cast<const uint4*>(v + o));
    }
#pragma unroll
    for (int i = 0; i < CP_ITERS; ++i) {
      if (src[i] < 0) continue;
      const int slot = slot0 + i * (CP_THREADS / 16);
      const int64_t o = ((int64_t)u * cap + slot) * row_bytes + c0;
      *reinterpret_cast<uint4*>((char*)c.k_cache + o) = kv[i];
      *reinterpret_cast<uint4*>((char*)c.v_cache + o) = vv[i];
    }
  }
  // per-slot decode state
  if (l16 == 0) {
#pragma unroll
    for (int i = 0; i < CP_ITERS; ++i) {
      const int slot = slot0 + i * (CP_THREADS / 16);
      if (slot >= cap) continue;
      const int64_t o = (int64_t)u * cap + slot;
      c.pos[o] = src[i];
      c.acc[o] = src[i] >= 0 ? __ldg(attn_acc + (int64_t)u * sh.T + src[i]) : 0.f;
      c.vnorm[o] = src[i] >= 0 ? __ldg(vnorm + (int64_t)u * sh.T + src[i]) : 0.f;
    }
  }
  }
  if (blockIdx.y == 0 && threadIdx.x == 0) {
    c.len[u] = len;
    c.free_slot[u] = len;
    c.next_pos[u] = sh.T;
    c.last_slot[u] = -1;
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
  static int sms = 0;
  if (!sms) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  }
  const int groups = (cap + CP_SLOTS - 1) / CP_SLOTS;
  int gy = 4 * sms / s.units;        // four CTAs fit on an SM
  gy = gy < 1 ? 1 : (gy > groups ? groups : gy);
  const dim3 grid(s.units, gy);
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
