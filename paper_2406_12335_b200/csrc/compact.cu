// KV compaction: gather the surviving K and V rows of every unit into the budgeted cache (bit-exact
// copies) and initialise the per-slot decode state.
//
// Pure data movement, so the rows never pass through registers: every warp owns a ring of shared-memory
// buffers; a batch is up to 16 consecutive destination slots of one unit.  Its K and V rows arrive by TMA
// row gathers (four rows per copy, indexed by the kept positions) when the inputs form one table of equally
// spaced rows, else by one bulk copy per row, all signalling one mbarrier; because the destination slots
// are consecutive, the batch then leaves with ONE bulk copy per tensor, shared -> global.  The next
// batches' rows are already in flight while a batch waits.
#include "vatp_internal.cuh"

namespace vatp {
namespace {

constexpr int CB_WARPS = 12;           // (with two batches in flight each: more warps with shallower rings beat 8 x 3 and 6 x 4)
constexpr int CB_THREADS = CB_WARPS * 32;
constexpr int CB_ROWS = 16;            // destination slots per batch at most (8 when the rows are 512 bytes)
constexpr int CB_MAXBUF = 4;           // batches in flight per warp (fewer when the rows are long)
constexpr size_t CB_SMEM = 196 * 1024;  // shared memory for the rings of a CTA
constexpr uint64_t CB_WAIT_NS = 1000000000ull;

__device__ __forceinline__ uint32_t cb_s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint64_t cb_now() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool cb_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(cb_s32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// bounded wait (about a second): false when the copies never signalled
__device__ __forceinline__ bool cb_wait(uint64_t* bar, uint32_t parity) {
  if (cb_try(bar, parity)) return true;
  const uint64_t t0 = cb_now();
  while (!cb_try(bar, parity))
    if (cb_now() - t0 > CB_WAIT_NS) return false;
  return true;
}

// One unit is cap slots = nb batches of 16 (the last one shorter); the batches of all units form one
// range that is split evenly over all warps of the grid, so that every SM moves the same number of bytes
// whatever the number of units or the budget.
// rows_pb: slots per batch.  gather_rs > 0: the inputs are tables of rows gather_rs elements apart that tm_k / tm_v
// describe, and full batches are fetched with four-row gathers.
__global__ void __launch_bounds__(CB_THREADS, 1)
compact_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, int64_t gather_rs,
               Shape sh, int elem_bytes, int B, int cap, const char* __restrict__ k, const char* __restrict__ v,
               const float* __restrict__ attn_acc, const float* __restrict__ vnorm, const int32_t* __restrict__ kept,
               vatp_cache c, int rows_pb, int nbuf, int32_t* dev_status) {
  extern __shared__ __align__(128) unsigned char cb_smem[];
  __shared__ __align__(8) uint64_t bars[CB_WARPS][CB_MAXBUF];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int row_bytes = sh.d * elem_bytes;
  const int buf_bytes = 2 * rows_pb * row_bytes;                 // K rows, then V rows
  unsigned char* my_buf = cb_smem + (size_t)wid * nbuf * buf_bytes;
  if (lane == 0) {
    for (int i = 0; i < CB_MAXBUF; ++i)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(cb_s32(&bars[wid][i])), "r"(1) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  // launched as a programmatic dependent of the selection: nothing is read before that has completed
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const int len = min(sh.T, B);
  const int nb = (cap + rows_pb - 1) / rows_pb;
  const int64_t total = (int64_t)sh.units * nb;
  const int64_t gw = (int64_t)blockIdx.x * CB_WARPS + wid, nw = (int64_t)gridDim.x * CB_WARPS;
  const int64_t b_begin = total * gw / nw, b_end = total * (gw + 1) / nw;
  const int64_t tok_bytes = sh.st * elem_bytes;
  const int l16 = lane & 15;
  const char* src_t = lane < 16 ? k : v;

  // request batch `bi` into ring slot `slot`: per-slot state is written on the way
  auto request = [&](int64_t bi, int slot) -> int {
    const int u = (int)(bi / nb);
    const int s0 = (int)(bi - (int64_t)u * nb) * rows_pb;
    const int s = s0 + l16;                                       // this lane's destination slot
    int src = -1;
    if (l16 < rows_pb && s < len) src = __ldg(kept + (int64_t)u * B + s);
    const int live = min(max(len - s0, 0), rows_pb);              // rows of the batch that hold a token
    uint64_t* bar = &bars[wid][slot];
    if (live > 0) {
      if (lane == 0)
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(cb_s32(bar)), "r"(2 * live * row_bytes) : "memory");
      __syncwarp();
      unsigned char* half = my_buf + (size_t)slot * buf_bytes + (lane < 16 ? 0 : rows_pb * row_bytes);
      bool gather = gather_rs > 0 && live == rows_pb;
#ifdef VATP_DEBUG_BOUNDS
      // the kept indices come from another kernel: a row outside the prompt, or a buffer offset outside the ring,
      // is not fetched (the batch's wait then runs out and is reported as well)
      if (src >= 0 && !VATP_INB(src, sh.T, dev_status)) src = -1;
      if (!VATP_INB((size_t)slot * buf_bytes + (lane < 16 ? 0 : rows_pb * row_bytes) + (l16 + 1) * row_bytes - 1,
                    (size_t)nbuf * buf_bytes, dev_status)) src = -1;
      gather = gather && __all_sync(0xffffffffu, src >= 0 || l16 >= rows_pb);
#endif
      if (gather) {
        // row index in the table of all rows; lanes 0-3 (K) and 16-19 (V) each gather four rows of the batch
        const int g = src >= 0 ? (int)((unit_offset(sh, u) + (int64_t)src * sh.st) / gather_rs) : 0;
        const int base_lane = (lane & 16) + 4 * (lane & 3);
        const int g0 = __shfl_sync(0xffffffffu, g, base_lane), g1 = __shfl_sync(0xffffffffu, g, base_lane + 1);
        const int g2 = __shfl_sync(0xffffffffu, g, base_lane + 2), g3 = __shfl_sync(0xffffffffu, g, base_lane + 3);
        if (l16 < rows_pb / 4)
          asm volatile(
              "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
              ::"r"(cb_s32(half + 4 * l16 * row_bytes)), "l"(reinterpret_cast<uint64_t>(lane < 16 ? &tm_k : &tm_v)),
                "r"(cb_s32(bar)), "r"(0), "r"(g0), "r"(g1), "r"(g2), "r"(g3)
              : "memory");
      } else if (src >= 0) {
        const char* from = src_t + unit_offset(sh, u) * elem_bytes + (int64_t)src * tok_bytes;
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(cb_s32(half + l16 * row_bytes)), "l"(from), "r"(row_bytes), "r"(cb_s32(bar)) : "memory");
      }
    }
    // per-slot decode state, and the unit's scalars with its first slot
    if (lane < rows_pb && s < cap && VATP_INB((int64_t)u * cap + s, (int64_t)sh.units * cap, dev_status)) {
      const int64_t o = (int64_t)u * cap + s;
      c.pos[o] = src;
      c.acc[o] = src >= 0 ? __ldg(attn_acc + (int64_t)u * sh.T + src) : 0.f;
      c.vnorm[o] = src >= 0 ? __ldg(vnorm + (int64_t)u * sh.T + src) : 0.f;
      if (s == 0) {
        c.len[u] = len;
        c.free_slot[u] = len;
        c.next_pos[u] = sh.T;
        c.last_slot[u] = -1;
      }
    }
    return live;
  };

  // Per ring slot: how many rows of its batch hold a token (8 bits each) and the parity of the barrier
  // phase that its copies complete (a batch of empty slots arms nothing).
  bool ok = true;
  uint32_t live_bits = 0, parity_bits = 0;
  const int64_t n_mine = b_end - b_begin;
  auto fill = [&](int64_t j) {            // batch j of this warp into ring slot j % nbuf
    const int slot = (int)(j % nbuf);
    const int live = request(b_begin + j, slot);
    live_bits = (live_bits & ~(0xffu << (8 * slot))) | ((uint32_t)live << (8 * slot));
  };
  for (int i = 0; i < nbuf && i < n_mine; ++i) fill(i);
  for (int64_t j = 0; j < n_mine; ++j) {
    const int slot = (int)(j % nbuf);
    const int64_t bi = b_begin + j;
    const int live = (int)((live_bits >> (8 * slot)) & 0xffu);
    if (live > 0) {
      if (ok && !cb_wait(&bars[wid][slot], (parity_bits >> slot) & 1u)) ok = false;
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      parity_bits ^= 1u << slot;
      if (lane == 0) {
        const int u = (int)(bi / nb);
        const int s0 = (int)(bi - (int64_t)u * nb) * rows_pb;
        const int64_t o = ((int64_t)u * cap + s0) * row_bytes;
        const unsigned char* from = my_buf + (size_t)slot * buf_bytes;
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                     ::"l"((char*)c.k_cache + o), "r"(cb_s32(from)), "r"(live * row_bytes) : "memory");
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                     ::"l"((char*)c.v_cache + o), "r"(cb_s32(from + rows_pb * row_bytes)), "r"(live * row_bytes) : "memory");
      }
    }
    if (lane == 0) asm volatile("cp.async.bulk.commit_group;" ::: "memory");      // (an empty group when nothing was live)
    // The ring slot of the batch before this one is requested again once its rows have been read out;
    // this batch's store stays in flight meanwhile.
    if (j >= 1 && j - 1 + nbuf < n_mine) {
      if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      __syncwarp();
      fill(j - 1 + nbuf);
    }
  }
  if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");       // shared memory outlives the copies
  if (!ok && lane == 0) {
    if (dev_status) atomicExch(dev_status, (int)VATP_ERR_TIMEOUT);
    // copies that were requested may still land: give each barrier one more bounded wait
    for (int i = 0; i < CB_MAXBUF; ++i) cb_wait(&bars[wid][i], (parity_bits >> i) & 1u);
  }
}

// Windowed indicator state: ring[u][(T - w + r) mod w][slot] = win_rows[u][r][kept[slot]] and the
// exact fixed-point window sum of every slot (Eq. 3).
__global__ void ring_kernel(int units, int T, int w, int B, int cap, const float* __restrict__ win_rows,
                            const int32_t* __restrict__ kept, vatp_cache c, int32_t* dev_status) {
  const int u = blockIdx.y;
  const int slot = blockIdx.x * blockDim.x + threadIdx.x;
  if (slot >= cap) return;
  const int len = min(T, B);
  int src = slot < len ? kept[(int64_t)u * B + slot] : -1;
  if (src >= 0 && !VATP_INB(src, T, dev_status)) src = -1;
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
                           int32_t* dev_status, cudaStream_t st) {
  const int eb = dtype == VATP_F32 ? 4 : 2;
  const int cap = cache_capacity(B);
  const int sms = device_sm_count();
  const int row_bytes = s.d * eb;
  const int rows_pb = row_bytes > 256 ? 8 : CB_ROWS;
  const int nb = (cap + rows_pb - 1) / rows_pb;
  const int64_t total = (int64_t)s.units * nb;
  const size_t per_buf = (size_t)CB_WARPS * 2 * rows_pb * row_bytes;     // one ring slot of every warp
  int nbuf = (int)(CB_SMEM / per_buf);
  nbuf = nbuf > CB_MAXBUF ? CB_MAXBUF : nbuf;
  if (nbuf < 2) return cudaErrorInvalidValue;                            // (head_dim <= 128 gives at least 2)
  const size_t smem = per_buf * nbuf;
  // Row gathers need the inputs as ONE table of equally spaced rows: the largest spacing that divides all three
  // strides (the row length itself for contiguous tensors and for [batch, T, heads, d] storage alike).
  auto gcd = [](int64_t a, int64_t b) { while (b) { const int64_t t = a % b; a = b; b = t; } return a; };
  int64_t rs = gcd(gcd(s.sb, s.sh), s.st);
  const int batch = s.units / s.heads;
  const int64_t last = (int64_t)(batch - 1) * s.sb + (int64_t)(s.heads - 1) * s.sh + (int64_t)(s.T - 1) * s.st;
  CUtensorMap tm_k = {}, tm_v = {};
  if (rs < s.d || (rs * eb) % 16 || last / rs >= ((int64_t)1 << 31) || !vatp_tc_available() ||
      !make_row_gather_map(&tm_k, k, (uint32_t)(row_bytes / 4), (uint64_t)(last / rs + 1), (uint64_t)(rs * eb)) ||
      !make_row_gather_map(&tm_v, v, (uint32_t)(row_bytes / 4), (uint64_t)(last / rs + 1), (uint64_t)(rs * eb)))
    rs = 0;                                                              // one bulk copy per row instead
  cudaError_t e = cudaFuncSetAttribute(compact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int64_t want = (total + CB_WARPS - 1) / CB_WARPS;          // at least one batch per warp
  const dim3 grid((unsigned)(want < sms ? want : sms));
  DependentLaunch dl(grid, dim3(CB_THREADS), smem, st);
  e = cudaLaunchKernelEx(&dl.cfg, compact_kernel, tm_k, tm_v, rs, s, eb, B, cap, (const char*)k, (const char*)v, attn_acc,
                         vnorm, kept, c, rows_pb, nbuf, dev_status);
  if (e != cudaSuccess) return e;
  if (s.window > 0 && win_rows) {
    ring_kernel<<<dim3((cap + 127) / 128, s.units), 128, 0, st>>>(s.units, s.T, s.window, B, cap, win_rows, kept, c, dev_status);
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace vatp
