// KV compaction: gather the surviving K and V rows of every unit into the budgeted cache with
// 16-byte loads and stores (bit-exact copies), and initialise the per-slot decode state.
#include "vatp_internal.cuh"

namespace vatp {
namespace {

constexpr int CP_THREADS = 256;
constexpr int CP_UNROLL = 4;

// One "chunk" is 16 bytes of one row of K or V.  Chunks are numbered
// ((unit * cap + slot) * 2 + which) * cpr + c, so consecutive threads copy consecutive 16-byte
// pieces of a row and a warp covers whole rows.
__global__ void __launch_bounds__(CP_THREADS)
compact_kernel(Shape sh, int elem_bytes, int B, int cap, const char* __restrict__ k, const char* __restrict__ v,
               const float* __restrict__ attn_acc, const float* __restrict__ vnorm, const int32_t* __restrict__ kept,
               vatp_cache c) {
  const int cpr = sh.d * elem_bytes / 16;  // chunks per row
  const int64_t total = (int64_t)sh.units * cap * 2 * cpr;
  const int len = min(sh.T, B);
  const int64_t base = ((int64_t)blockIdx.x * CP_UNROLL) * CP_THREADS + threadIdx.x;
  uint4 val[CP_UNROLL];
  int64_t dst[CP_UNROLL];
#pragma unroll
  for (int it = 0; it < CP_UNROLL; ++it) {
    const int64_t idx = base + (int64_t)it * CP_THREADS;
    dst[it] = -1;
    if (idx >= total) continue;
    const int cc = (int)(idx % cpr);
    const int64_t row = idx / cpr;
    const int which = (int)(row & 1);
    const int64_t us = row >> 1;
    const int slot = (int)(us % cap);
    const int u = (int)(us / cap);
    const int src = slot < len ? kept[(int64_t)u * B + slot] : -1;
    if (cc == 0 && which == 0) {
      const int64_t o = (int64_t)u * cap + slot;
      c.pos[o] = src;
      c.acc[o] = src >= 0 ? attn_acc[(int64_t)u * sh.T + src] : 0.f;
      c.vnorm[o] = src >= 0 ? vnorm[(int64_t)u * sh.T + src] : 0.f;
      if (slot == 0) {
        c.len[u] = len;
        c.free_slot[u] = len;
        c.next_pos[u] = sh.T;
      }
    }
    if (src < 0) continue;
    const char* in = (which ? v : k) + (unit_offset(sh, u) + (int64_t)src * sh.st) * elem_bytes + (int64_t)cc * 16;
    val[it] = *reinterpret_cast<const uint4*>(in);
    dst[it] = (((int64_t)u * cap + slot) * cpr + cc) * 16;
    if (which) dst[it] = -2 - dst[it];  // tag V destinations
  }
#pragma unroll
  for (int it = 0; it < CP_UNROLL; ++it) {
    if (dst[it] == -1) continue;
    if (dst[it] >= 0)
      *reinterpret_cast<uint4*>((char*)c.k_cache + dst[it]) = val[it];
    else
      *reinterpret_cast<uint4*>((char*)c.v_cache + (-2 - dst[it])) = val[it];
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
  const int cpr = s.d * eb / 16;
  const int64_t total = (int64_t)s.units * cap * 2 * cpr;
  const int64_t per_block = (int64_t)CP_THREADS * CP_UNROLL;
  const unsigned blocks = (unsigned)((total + per_block - 1) / per_block);
  compact_kernel<<<blocks, CP_THREADS, 0, st>>>(s, eb, B, cap, (const char*)k, (const char*)v, attn_acc, vnorm, kept, c);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (s.window > 0) {
    ring_kernel<<<dim3((cap + 127) / 128, s.units), 128, 0, st>>>(s.units, s.T, s.window, B, cap, win_rows, kept, c);
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace vatp
