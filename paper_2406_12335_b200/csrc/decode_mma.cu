// Decode step for bf16, head_dim 128 (the LLaMA2-7B shape): append, attend (Eq. 1), indicator
// update (Eq. 2 / Eq. 3), importance (Eq. 4), release of the lowest-importance unprotected slot.
//
// The step is HBM-bound (every cached K and V row is read once) but so short - tens of megabytes -
// that fixed latencies decide its duration.  Hence:
//   * every warp owns a ring of stages and requests its first stages (tiled TMA loads of 16 rows x
//     128 bytes, 128-byte swizzled so that ldmatrix is conflict-free) before anything else happens;
//   * q.K^T and p.V run on the warp-level tensor-core path (mma.sync m16n8k16, bf16 in, fp32
//     accumulate): S^T = q K^T leaves the probabilities of 16 rows in exactly the registers the
//     A operand of p V wants, so a 16-row group costs about 80 instructions.  p is split into two
//     bf16 halves (rows 0-7 / 8-15 of the A tile carry hi / lo): the product keeps ~16 bits of p;
//   * a unit is split over a thread-block cluster when units are few.  Every CTA PUSHES its running
//     max and sum into the shared memory of all CTAs of the unit and its partial output into rank
//     0's; after one cluster barrier each CTA knows the softmax normaliser, updates the indicators of
//     its own slots and proposes its own eviction candidate to rank 0; after a second barrier rank 0
//     picks the candidate of the whole unit.  No global scratch, one launch;
//   * consecutive steps overlap (programmatic dependent launch).  By default a step requests its
//     first K/V tiles early and reads everything else only after all earlier work in the stream has
//     completed; its control warp releases the next launch once that wait is over, so at most one
//     unfinished predecessor exists while a step sets up, and the one cache row that predecessor
//     may have written - the row of its incoming token, recorded in last_slot - is re-read after
//     the wait and patched in.  A caller that steps several independent caches on one stream may
//     opt in (VATP_FLAG_DECODE_OVERLAP) to more: the host keeps, per stream, the buffers of the
//     last launches, and a launch that shares no buffer with any launch that can still be in
//     flight (another layer's or another sequence's cache) never waits: its control warp releases
//     the next launch at once and only holds the CTA until the previous launch has completed, so
//     launches still complete in order and the number in flight is bounded by what fits on the
//     machine (two CTAs fit on an SM).  A launch that does wait has its SMs to itself and runs the
//     eight-warp variant of the kernel (same arithmetic, see MW below);
//   * grouped-query attention (several query heads share one cache; the paper leaves the case open and points at
//     a group-wise score, read here as the MEAN of the heads' probabilities): up to eight heads of a group ride
//     in the rows of the MMA tiles (template parameter GT), so a K or V row is still read once per step.
#include <cooperative_groups.h>

#include <mutex>

#include "vatp_internal.cuh"

namespace cg = cooperative_groups;

namespace vatp {
namespace {

// Streaming warps per CTA (template parameter MW of the kernel; their threads WT = 32 MW, plus one control warp):
// four when launches of different caches run side by side (two CTAs per SM), eight for a launch that waits for its
// predecessor and has the SM to itself - one warp per scheduler cannot hide the latency of its own
// ldmatrix / mma.sync / softmax chain, so such a launch streams faster with two.
// The arithmetic does not depend on MW: a CTA's 16-row groups are always dealt to NSTREAM = 8 online-softmax streams -
// the groups below the midpoint H (a multiple of four) to streams 0-3 by g mod 4, those from H on to streams 4-7 -
// each stream is folded in ascending group order, and the eight partials are merged in stream order.  A warp of the
// eight-warp kernel folds one stream; warp w of the four-warp kernel walks groups w, w + 4, ... in one sweep,
// files its partial under stream w where it crosses H and starts afresh for stream w + 4.  Results are
// bit-identical whichever kernel a launch gets.
constexpr int MW_BESIDE = 4, MW_ALONE = 8;
constexpr int NSTREAM = 8;
constexpr int HD = 128;
constexpr int GROUP = 16;             // rows per MMA group = rows of K (and of V) per stage
constexpr int ROW_BYTES = HD * 2;
constexpr int TILE_BYTES = GROUP * 128;    // 16 rows x 64 bf16, 128-byte swizzled
constexpr int STAGE_BYTES = 4 * TILE_BYTES; // K columns 0-63, K 64-127, V 0-63, V 64-127
constexpr int MAX_SPLIT = 8;
constexpr int GQ_HEADS = 8;           // grouped queries: query heads per cache this kernel takes (rows 0-7 of the MMA tiles)
constexpr int GQ_MAX_SPLIT = MAX_SPLIT;   // ... and the CTAs a unit is split over at most
constexpr float LOG2E = 1.4426950408889634f;
constexpr unsigned long long NO_KEY = ~0ull;

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
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// two floats -> packed bf16 pair (lo in the low half), round to nearest
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// barrier over the streaming warps only (the control warp does not take part)
template <int WT>
__device__ __forceinline__ void workers_sync() { asm volatile("bar.sync 1, %0;" ::"n"(WT) : "memory"); }
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// what the CTAs of a unit push into one another
struct Exch {
  float m[MAX_SPLIT], l[MAX_SPLIT];       // in every rank: per rank the max of its logits (log2 domain) and the sum of exp2(s - m)
  float o[MAX_SPLIT][HD];                 // in rank 0: partial outputs of every rank
  unsigned long long key[MAX_SPLIT];      // in rank 0: every rank's eviction candidate (NO_KEY: none) ...
  int key_slot[MAX_SPLIT], key_pos[MAX_SPLIT];   // ... its slot in the unit and its position
};


// eviction order as one integer: lower importance first, among equals the higher position first
__device__ __forceinline__ unsigned long long evict_key(float I, int pos) {
  return ((unsigned long long)__float_as_uint(I) << 32) | (unsigned)(0x7fffffff - pos);
}
// minimum of a 64-bit key over the warp, in two 32-bit steps
__device__ __forceinline__ unsigned long long warp_min_key(unsigned long long key) {
  const unsigned h = (unsigned)(key >> 32);
  const unsigned mh = __reduce_min_sync(0xffffffffu, h);
  const unsigned ml = __reduce_min_sync(0xffffffffu, h == mh ? (unsigned)key : 0xffffffffu);
  return ((unsigned long long)mh << 32) | ml;
}

// GT = 1: one query head per cache (multi-head attention).  GT = GQ_HEADS: grouped queries - up to GQ_HEADS query
// heads (G of them, a run-time argument) share the cache of unit u: row g of the MMA tiles carries head g, so the
// streaming loop is the same instructions, and every K and V row is read once for the whole group; the maxima,
// sums and partial outputs exist per head, and the indicator advances by the MEAN of the heads' probabilities.
// Only the eight-warp kernel is built for it (the per-head partials take the room a second CTA would need).
template <bool WINDOWED, int MW, int GT>
__global__ void __launch_bounds__(MW * 32 + 32, MW == MW_BESIDE ? 2 : 1)
decode_mma_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, int independent, int G,
                  int state_in_smem, int split, int chunk, int nstage, int B, int cap, int F, int R, int w, int norm, float scale_log2,
                  vatp_cache c,
                  const __nv_bfloat16* __restrict__ q_new, const __nv_bfloat16* __restrict__ k_new,
                  const __nv_bfloat16* __restrict__ v_new, __nv_bfloat16* __restrict__ out,
                  int32_t* __restrict__ evicted, int32_t* __restrict__ dev_status) {
  constexpr int WT = MW * 32;           // streaming threads (at least HD: one per output channel where outputs are formed)
  static_assert(WT >= HD, "one streaming thread per output channel");
  static_assert(GT == 1 || (GT == GQ_HEADS && MW == MW_ALONE), "grouped queries: the eight-warp kernel only");
  extern __shared__ unsigned char dyn_raw[];
  unsigned char* dyn = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(dyn_raw) + 1023) & ~uintptr_t(1023));
  // [MW][nstage] stages | logits[chunk] | acc[chunk] | vnorm[chunk] | pos[chunk]: the per-slot arrays of
  // this CTA's own slots.  For large caches only the logits are held here, which keeps the CTA small
  // enough for two launches to be resident together; acc, vnorm and pos are then copied into the stage
  // memory once the streaming is over (state_in_smem == 2) or, if even that is too small, read from
  // global memory in the tail (state_in_smem == 0).
  unsigned char* stage_base = dyn;
  float* logit_s = reinterpret_cast<float*>(dyn + (size_t)MW * nstage * STAGE_BYTES);
  // (grouped queries: logits[G][chunk], state always here (state_in_smem == 1), then the per-head partial outputs
  // of the eight streams [NSTREAM][G][HD] and, in rank 0, those of every CTA of the unit [split][G][HD])
  float* acc_s = state_in_smem == 2 ? reinterpret_cast<float*>(stage_base) : logit_s + (GT > 1 ? G : 1) * chunk;
  float* vn_s = acc_s + chunk;
  int* pos_s = reinterpret_cast<int*>(vn_s + chunk);
  float* gq_part = reinterpret_cast<float*>(pos_s + chunk);
  float* gq_xo = gq_part + NSTREAM * (GT > 1 ? G : 0) * HD;

  __shared__ __align__(8) uint64_t bars[MW * 4 + 1];
  __shared__ __align__(16) Exch ex;
  constexpr int SPW = NSTREAM / MW;     // streams per warp
  static_assert(SPW == 1 || SPW == 2, "a warp folds one or two streams");
  __shared__ __align__(16) float part_o[NSTREAM][HD];
  __shared__ float part_m[NSTREAM], part_l[NSTREAM];
  // grouped queries: per stream and head; per rank and head (pushed by every CTA of the unit); the unit's normalisers
  __shared__ float gq_pm[GT > 1 ? NSTREAM : 1][GT], gq_pl[GT > 1 ? NSTREAM : 1][GT];
  __shared__ float gq_m[GT > 1 ? GQ_MAX_SPLIT : 1][GT], gq_l[GT > 1 ? GQ_MAX_SPLIT : 1][GT];
  __shared__ float gq_fr[GT > 1 ? GQ_MAX_SPLIT : 1][GT], gq_mall[GT], gq_invl[GT];
  __shared__ unsigned long long warp_key[MW];
  __shared__ int ctrl_evicting;

  cg::cluster_group cluster = cg::this_cluster();
  const int rank = split > 1 ? (int)cluster.block_rank() : 0;
  const int u = blockIdx.x / split;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int j4 = lane & 3;

  // Remote shared memory may only be touched once its CTA runs: everyone arrives here, and waits
  // (long since satisfied) just before the first remote store.
  if (split > 1) asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");   // all five warps

  if (wid == MW) {
    // ---- control warp: release the next launch, then hold this CTA until the previous launch has completed
    // (it arrives at the unit's barrier at once, so that the streaming warps never wait for it)
    // (its arrivals at the unit's two barriers come as early as the barrier's phases allow)
    if (split > 1) { cluster_wait_acquire(); cluster_arrive_release(); }
    if (lane == 0) {
      // An independent launch lets its successor start at once.  A launch that waits for its
      // predecessor releases its successor only after that wait: the successor's early tile
      // requests then race with this launch alone, never with launches before it.
      if (independent) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
      asm volatile("griddepcontrol.wait;" ::: "memory");
      if (!independent) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    __syncwarp();
    if (split > 1) {
      cluster_wait_acquire();
      // a second barrier follows when the step evicts (the streaming warps have published that by now)
      if (*reinterpret_cast<volatile int*>(&ctrl_evicting)) { cluster_arrive_release(); cluster_wait_acquire(); }
    }
    return;
  }

  // this CTA's slot range inside the allocation
  const int s0 = min(rank * chunk, cap);
  const int rows_alloc = min(chunk, cap - s0);
  const int ngroups = (rows_alloc + GROUP - 1) / GROUP;
  const int row_base = u * cap + s0;     // first row of the range in the [units * cap, 128] view of the caches
  uint64_t* my_bars = &bars[wid * 4];
  uint64_t* state_bar = &bars[MW * 4];
  unsigned char* my_stages = stage_base + (size_t)wid * nstage * STAGE_BYTES;

  // every warp arms its own barriers: no CTA-wide barrier before the first copy is requested
  if (lane == 0) {
    for (int s = 0; s < nstage; ++s) mbar_init(&my_bars[s], 1);
    if (wid == 1) mbar_init(state_bar, 1);     // armed and used by this same lane
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  // lanes 0-3 fetch the four tiles of group g (rows beyond the caches arrive as zeros)
  auto issue = [&](int g, int stage) {
    unsigned char* dst = my_stages + stage * STAGE_BYTES;
    uint64_t* bar = &my_bars[stage];
    if (lane == 0) mbar_expect_tx(bar, STAGE_BYTES);
    __syncwarp();
    if (lane < 4) tma_load_2d(dst + lane * TILE_BYTES, lane < 2 ? &tm_k : &tm_v, bar, (lane & 1) * 64, row_base + g * GROUP);
  };
  // This warp's groups: g_first, g_first + 4, ... below g_end.  H: where streams 4-7 begin.
  const int H = ((ngroups + 7) >> 3) << 2;
  const int g_first = SPW == 2 ? wid : (wid < 4 ? wid : H + wid - 4);
  const int g_end = (SPW == 2 || wid >= 4) ? ngroups : min(H, ngroups);
  for (int s = 0; s < nstage; ++s)
    if (g_first + s * 4 < g_end) issue(g_first + s * 4, s);
  // The next launch in the stream may start now; nothing below this line is read before the previous
  // launch has completed and its writes are visible.
  if (!independent) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tid == 32 && rows_alloc > 0) {      // per-slot state of this CTA's slots
    const int64_t o = (int64_t)u * cap + s0;
    if (state_in_smem == 1) {
      mbar_expect_tx(state_bar, 3u * rows_alloc * 4u);
      bulk_g2s(acc_s, c.acc + o, rows_alloc * 4, state_bar);
      bulk_g2s(vn_s, c.vnorm + o, rows_alloc * 4, state_bar);
      bulk_g2s(pos_s, c.pos + o, rows_alloc * 4, state_bar);
    } else if (state_in_smem == 0) {
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(c.acc + o), "r"(rows_alloc * 4) : "memory");
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(c.vnorm + o), "r"(rows_alloc * 4) : "memory");
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(c.pos + o), "r"(rows_alloc * 4) : "memory");
    }
  }

  const int len = c.len[u];
  const int fs = c.free_slot[u];
  const int t = c.next_pos[u];
  const int ls = c.last_slot[u];
#ifdef VATP_DEBUG_BOUNDS
  // the state words come from memory: out of range, nothing of this unit is touched
  if (!VATP_INB(len, cap, dev_status) || !VATP_INB(fs, cap, dev_status) || !VATP_INB(ls + 1, cap + 1, dev_status)) {
    if (tid == 0) ctrl_evicting = 0;
    if (split > 1) {      // the unit's first barrier is still reached by every thread (all its CTAs read the same words)
      cluster_wait_acquire();
      cluster_arrive_release(); cluster_wait_acquire();
    }
    return;
  }
#endif
  const int hi = len + 1;                // slots [0, hi) are live once the new token is in
  const int cnt = max(min(hi - s0, rows_alloc), 0);
  const int fs_local = fs - s0;          // row of the incoming token inside this CTA's range (if owned)
  const bool owns_new = fs_local >= 0 && fs_local < cnt;
  if (WINDOWED && tid == 64 && rows_alloc > 0) {
    // the tail reads the ring row that leaves the window and the exact sums: have them in L2 by then
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(c.ring + ((int64_t)u * w + (t % w)) * cap + s0), "r"(rows_alloc * 4) : "memory");
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(c.acc_fixed + (int64_t)u * cap + s0), "r"(rows_alloc * 8) : "memory");
  }
  if (tid == 0) ctrl_evicting = hi > B ? 1 : 0;     // read by the control warp after the first barrier
  const int ls_local = ls - s0;          // row the previous step appended (its tile may predate that store)
  const bool owns_last = !independent && ls >= 0 && ls != fs && ls_local >= 0 && ls_local < cnt;

  // A operand of q K^T: q replicated over the rows 0-7 of the tile (rows 8-15 zero)
  // (grouped queries: row g of the tile carries head g of the unit's group; rows beyond the group repeat its last head)
  const __nv_bfloat16* qn = GT > 1 ? q_new + ((int64_t)u * G + min(lane >> 2, G - 1)) * HD : q_new + (int64_t)u * HD;
  uint32_t qa[HD / 16][2];
#pragma unroll
  for (int ks = 0; ks < HD / 16; ++ks) {
    qa[ks][0] = __ldg(reinterpret_cast<const uint32_t*>(qn + ks * 16 + 2 * j4));
    qa[ks][1] = __ldg(reinterpret_cast<const uint32_t*>(qn + ks * 16 + 8 + 2 * j4));
  }
  // 16 bytes of the incoming K row (lanes 0-15) or V row (lanes 16-31)
  const uint4 new_raw = __ldg(reinterpret_cast<const uint4*>((lane < 16 ? k_new : v_new) + (int64_t)u * HD) + (lane & 15));

  uint4 last_raw = make_uint4(0u, 0u, 0u, 0u);
  if (owns_last)
    last_raw = *(reinterpret_cast<const uint4*>((const __nv_bfloat16*)(lane < 16 ? c.k_cache : c.v_cache) +
                                                ((int64_t)u * cap + ls) * HD) + (lane & 15));

  // ---- append: the CTA that owns the free slot stores the new row and its norm (Eq. 4) ----
  float new_norm = 0.f;
  {
    const uint32_t wv[4] = {new_raw.x, new_raw.y, new_raw.z, new_raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
      new_norm = norm_fold(norm, norm_fold(norm, new_norm, __uint_as_float(wv[i] << 16)), __uint_as_float(wv[i] & 0xffff0000u));
#pragma unroll
    for (int o = 8; o; o >>= 1) new_norm = norm_merge(norm, new_norm, __shfl_xor_sync(0xffffffffu, new_norm, o));
    new_norm = norm_finish(norm, __shfl_sync(0xffffffffu, new_norm, 16));      // the V half's partial
  }
  if (owns_new && wid == 0) {
    __nv_bfloat16* dst = (__nv_bfloat16*)(lane < 16 ? c.k_cache : c.v_cache) + ((int64_t)u * cap + fs) * HD;
    reinterpret_cast<uint4*>(dst)[lane & 15] = new_raw;
    if (lane == 0) {
      c.vnorm[(int64_t)u * cap + fs] = new_norm;
      c.pos[(int64_t)u * cap + fs] = t;
    }
  }
  if (split > 1) cluster_wait_acquire();

  // ---- stream the groups: logits, online softmax, partial output ----
  float m_run = -INFINITY, l_run = 0.f;
  float o_acc[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) { o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f; }
  bool ok = true;
  // ldmatrix lane addressing: matrix i = lane / 8, row r = lane % 8.  A tile row is 128 bytes and its
  // 16-byte chunk c sits at position c ^ (row % 8).
  //   K (plain):  matrices (rows 0-7, k lo), (rows 0-7, k hi), (rows 8-15, k lo), (rows 8-15, k hi)
  //   V (trans):  matrices (rows 0-7, n lo), (rows 8-15, n lo), (rows 0-7, n hi), (rows 8-15, n hi)
  const int lm_i = lane >> 3, lm_r = lane & 7;
  const uint32_t k_row_off = (uint32_t)(((lm_i >> 1) * 8 + lm_r) * 128), k_x = (uint32_t)((lm_i & 1) ^ lm_r);
  const uint32_t v_row_off = (uint32_t)(((lm_i & 1) * 8 + lm_r) * 128), v_x = (uint32_t)((lm_i >> 1) ^ lm_r);
  // the running partial goes to its stream's slot (every lane with the same j4 holds the same values; rows 0-7
  // are the hi part, 8-15 the lo part)
  auto flush = [&](int stream) {
    float l = l_run;
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if constexpr (GT > 1) {
      const int hg = lane >> 2;      // this lane's head
      if (hg < G) {
        float* po = gq_part + ((size_t)stream * G + hg) * HD;
#pragma unroll
        for (int i = 0; i < HD / 8; ++i)
          *reinterpret_cast<float2*>(&po[i * 8 + 2 * j4]) = make_float2(o_acc[i][0] + o_acc[i][2], o_acc[i][1] + o_acc[i][3]);
        if (j4 == 0) { gq_pm[stream][hg] = m_run; gq_pl[stream][hg] = l; }
      }
    } else if (lane < 4) {
#pragma unroll
      for (int i = 0; i < HD / 8; ++i)
        *reinterpret_cast<float2*>(&part_o[stream][i * 8 + 2 * j4]) = make_float2(o_acc[i][0] + o_acc[i][2], o_acc[i][1] + o_acc[i][3]);
      if (lane == 0) { part_m[stream] = m_run; part_l[stream] = l; }
    }
  };
  int it = 0, g = g_first;
  bool past_live = false, second = false;
  // folds this warp's groups below g_stop into the running partial
  auto fold_groups = [&](int g_stop) {
    for (; g < g_stop; g += 4, ++it) {
      if (it >= nstage && g * GROUP >= cnt) { past_live = true; break; }     // never requested (see the end of the loop body)
      const int stage = it % nstage;
      const uint32_t parity = (it / nstage) & 1;
      if (ok && !mbar_wait(&my_bars[stage], parity)) ok = false;
      ok = __all_sync(0xffffffffu, ok);
      unsigned char* ks = my_stages + stage * STAGE_BYTES;
      unsigned char* vs = ks + 2 * TILE_BYTES;
      const int r0 = g * GROUP;
      bool wrote = false;
      if (ok && r0 < cnt) {
        // the incoming token's row is not in the cache yet: patch it in; rows beyond the live range
        // must not reach the p V product (their probability is 0, but 0 * garbage need not be 0)
        if (owns_new && fs_local >= r0 && fs_local < r0 + GROUP) {
          const int rr = fs_local - r0, ch = lane & 15;
          *reinterpret_cast<uint4*>((lane < 16 ? ks : vs) + (ch >> 3) * TILE_BYTES + rr * 128 + (((ch & 7) ^ (rr & 7)) << 4)) = new_raw;
          wrote = true;
        }
        if (owns_last && ls_local >= r0 && ls_local < r0 + GROUP) {
          const int rr = ls_local - r0, ch = lane & 15;
          *reinterpret_cast<uint4*>((lane < 16 ? ks : vs) + (ch >> 3) * TILE_BYTES + rr * 128 + (((ch & 7) ^ (rr & 7)) << 4)) = last_raw;
          wrote = true;
        }
        if (cnt < r0 + GROUP) {
          for (int rr = cnt - r0 + (lane >> 4); rr < GROUP; rr += 2)
            *reinterpret_cast<uint4*>(vs + ((lane >> 3) & 1) * TILE_BYTES + rr * 128 + ((lane & 7) << 4)) = make_uint4(0u, 0u, 0u, 0u);
          wrote = true;
        }
        __syncwarp();
        // S^T = q K^T: two n-tiles of 8 rows; c[0], c[1] = logits of rows 2 j4, 2 j4 + 1 of the tile
        float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t kaddr = smem_u32(ks) + k_row_off;
  #pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          uint32_t bf[4];
          ldsm_x4(kaddr + (kk >> 2) * TILE_BYTES + ((k_x ^ ((2 * kk) & 7)) << 4), bf);
          mma_bf16(sa, qa[kk][0], 0u, qa[kk][1], 0u, bf[0], bf[1]);
          mma_bf16(sb, qa[kk][0], 0u, qa[kk][1], 0u, bf[2], bf[3]);
        }
        float s[4] = {sa[0] * scale_log2, sa[1] * scale_log2, sb[0] * scale_log2, sb[1] * scale_log2};
        const int rows[4] = {r0 + 2 * j4, r0 + 2 * j4 + 1, r0 + 8 + 2 * j4, r0 + 9 + 2 * j4};
  #pragma unroll
        for (int i = 0; i < 4; ++i)
          if (rows[i] >= cnt) s[i] = -INFINITY;
        if constexpr (GT > 1) {
          if ((lane >> 2) < G) {
  #pragma unroll
            for (int i = 0; i < 4; ++i)
              if (rows[i] < cnt) logit_s[(lane >> 2) * chunk + rows[i]] = s[i];
          }
        } else if (lane < 4) {
  #pragma unroll
          for (int i = 0; i < 4; ++i)
            if (rows[i] < cnt) logit_s[rows[i]] = s[i];
        }
        float gmax = fmaxf(fmaxf(s[0], s[1]), fmaxf(s[2], s[3]));
        gmax = fmaxf(gmax, __shfl_xor_sync(0xffffffffu, gmax, 1));
        gmax = fmaxf(gmax, __shfl_xor_sync(0xffffffffu, gmax, 2));
        if (gmax > m_run) {          // uniform over a tile row's four lanes - over the warp with one head (r0 < cnt guarantees a live row, so gmax is finite)
          const float f = ex2(m_run - gmax);   // 0 on the first group
          l_run *= f;
  #pragma unroll
          for (int i = 0; i < HD / 8; ++i) { o_acc[i][0] *= f; o_acc[i][1] *= f; o_acc[i][2] *= f; o_acc[i][3] *= f; }
          m_run = gmax;
        }
        float p[4];
  #pragma unroll
        for (int i = 0; i < 4; ++i) { p[i] = ex2(s[i] - m_run); l_run += p[i]; }
        // A operand of p V: rows 0-7 carry the high bf16 half of p, rows 8-15 the remainder
        const uint32_t hi0 = pack_bf16(p[0], p[1]), hi1 = pack_bf16(p[2], p[3]);
        const uint32_t lo0 = pack_bf16(p[0] - __uint_as_float(hi0 << 16), p[1] - __uint_as_float(hi0 & 0xffff0000u));
        const uint32_t lo1 = pack_bf16(p[2] - __uint_as_float(hi1 << 16), p[3] - __uint_as_float(hi1 & 0xffff0000u));
        const uint32_t vaddr = smem_u32(vs) + v_row_off;
  #pragma unroll
        for (int nn = 0; nn < HD / 16; ++nn) {
          uint32_t bf[4];
          ldsm_x4_t(vaddr + (nn >> 2) * TILE_BYTES + ((v_x ^ ((2 * nn) & 7)) << 4), bf);
          mma_bf16(o_acc[2 * nn], hi0, lo0, hi1, lo1, bf[0], bf[1]);
          mma_bf16(o_acc[2 * nn + 1], hi0, lo0, hi1, lo1, bf[2], bf[3]);
        }
      }
      // generic-proxy stores into a stage must be ordered before the next bulk copy into it
      if (wrote) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      const int next = g + nstage * 4;
      // later requests know the live range: groups beyond it are not fetched
      if (ok && next < g_end && next * GROUP < cnt) issue(next, stage);
    }
  };
  if (SPW == 2) {
    // the four-warp kernel: stream wid up to the midpoint, filed, then stream wid + 4 from a fresh partial
    fold_groups(min(H, g_end));
    if (!past_live && g < g_end) {
      flush(wid);
      second = true;
      m_run = -INFINITY;
      l_run = 0.f;
#pragma unroll
      for (int i = 0; i < HD / 8; ++i) { o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f; }
      fold_groups(g_end);
    }
  } else {
    fold_groups(g_end);
  }
  if (!ok && lane == 0) {
    // a copy never completed: flag it and give what is still in flight one more bounded wait
    if (dev_status) atomicExch(dev_status, (int)VATP_ERR_TIMEOUT);
    for (int s = 0; s < nstage; ++s) mbar_wait(&my_bars[s], 0);
  }
  flush(second ? wid + MW : wid);
  if (SPW == 2 && !second) {      // the four-warp kernel never reached the midpoint: its stream wid + 4 is empty
    *reinterpret_cast<float4*>(&part_o[wid + MW][lane * 4]) = make_float4(0.f, 0.f, 0.f, 0.f);
    if (lane == 0) { part_m[wid + MW] = -INFINITY; part_l[wid + MW] = 0.f; }
  }
  workers_sync<WT>();
  if (state_in_smem == 2 && tid == 32 && rows_alloc > 0) {
    // every stage of this CTA has been consumed: the per-slot state of its slots lands there while the
    // cluster gathers (the stages were last written by bulk copies and read by ldmatrix; warps that
    // stored into them have fenced)
    const int64_t o = (int64_t)u * cap + s0;
    mbar_expect_tx(state_bar, 3u * rows_alloc * 4u);
    bulk_g2s(acc_s, c.acc + o, rows_alloc * 4, state_bar);
    bulk_g2s(vn_s, c.vnorm + o, rows_alloc * 4, state_bar);
    bulk_g2s(pos_s, c.pos + o, rows_alloc * 4, state_bar);
  }

  // ---- CTA partial: max and sum to every CTA of the unit, partial output to rank 0 ----
  if constexpr (GT > 1) {
    // per head of the group; thread tid < HD merges channel tid of the eight streams, threads HD .. HD + split - 1
    // push the head's maximum and sum to the unit's CTAs
    float* xo0 = split > 1 ? cluster.map_shared_rank(gq_xo, 0) : gq_xo;
    for (int h = 0; h < G; ++h) {
      float m_c = -INFINITY;
#pragma unroll
      for (int i = 0; i < NSTREAM; ++i) m_c = fmaxf(m_c, gq_pm[i][h]);
      float fw[NSTREAM], l_c = 0.f;
#pragma unroll
      for (int i = 0; i < NSTREAM; ++i) {
        fw[i] = gq_pm[i][h] > -INFINITY ? ex2(gq_pm[i][h] - m_c) : 0.f;
        l_c += gq_pl[i][h] * fw[i];
      }
      if (tid < HD) {
        float a = 0.f;
#pragma unroll
        for (int i = 0; i < NSTREAM; ++i) a = fmaf(gq_part[((size_t)i * G + h) * HD + tid], fw[i], a);
        xo0[((size_t)rank * G + h) * HD + tid] = a;
      } else if (tid < HD + split) {
        const int r = tid - HD;
        float* rm = split > 1 ? cluster.map_shared_rank(&gq_m[0][0], r) : &gq_m[0][0];
        float* rl = split > 1 ? cluster.map_shared_rank(&gq_l[0][0], r) : &gq_l[0][0];
        rm[rank * GT + h] = m_c;
        rl[rank * GT + h] = l_c;
      }
    }
  } else {
    float m_c = -INFINITY;
#pragma unroll
    for (int i = 0; i < NSTREAM; ++i) m_c = fmaxf(m_c, part_m[i]);
    float fw[NSTREAM], l_c = 0.f;
#pragma unroll
    for (int i = 0; i < NSTREAM; ++i) {
      fw[i] = part_m[i] > -INFINITY ? ex2(part_m[i] - m_c) : 0.f;
      l_c += part_l[i] * fw[i];
    }
    Exch* e0 = split > 1 ? cluster.map_shared_rank(&ex, 0) : &ex;
    if (tid < HD) {
      float a = 0.f;
#pragma unroll
      for (int i = 0; i < NSTREAM; ++i) a = fmaf(part_o[i][tid], fw[i], a);
      e0->o[rank][tid] = a;
    }
    if (tid < split) {
      Exch* er = split > 1 ? cluster.map_shared_rank(&ex, tid) : &ex;
      er->m[rank] = m_c;
      er->l[rank] = l_c;
    }
  }
  if (split > 1) { cluster_arrive_release(); cluster_wait_acquire(); } else workers_sync<WT>();

  // ---- every CTA: the unit's softmax normaliser (all data is local now) ----
  if constexpr (GT > 1) {
    if (tid < G) {         // one thread per head
      float m_h = -INFINITY, L_h = 0.f;
      for (int r = 0; r < split; ++r) m_h = fmaxf(m_h, gq_m[r][tid]);
      for (int r = 0; r < split; ++r) {
        const float f = gq_m[r][tid] > -INFINITY ? ex2(gq_m[r][tid] - m_h) : 0.f;
        gq_fr[r][tid] = f;
        L_h += gq_l[r][tid] * f;
      }
      gq_mall[tid] = m_h;
      gq_invl[tid] = 1.f / L_h;
    }
    workers_sync<WT>();
    if (rank == 0 && tid < HD) {
      for (int h = 0; h < G; ++h) {
        float a = 0.f;
        for (int r = 0; r < split; ++r) a = fmaf(gq_xo[((size_t)r * G + h) * HD + tid], gq_fr[r][h], a);
        out[((int64_t)u * G + h) * HD + tid] = __float2bfloat16(a * gq_invl[h]);
      }
    }
  }
  float m_all = -INFINITY, L = 0.f;
  float fr[MAX_SPLIT];
#pragma unroll
  for (int r = 0; r < MAX_SPLIT; ++r)
    if (r < split) m_all = fmaxf(m_all, ex.m[r]);
#pragma unroll
  for (int r = 0; r < MAX_SPLIT; ++r) {
    fr[r] = (r < split && ex.m[r] > -INFINITY) ? ex2(ex.m[r] - m_all) : 0.f;
    if (r < split) L += ex.l[r] * fr[r];
  }
  const float invL = 1.f / L;
  if (GT == 1 && rank == 0 && tid < HD) {
    float a = 0.f;
#pragma unroll
    for (int r = 0; r < MAX_SPLIT; ++r)
      if (r < split) a = fmaf(ex.o[r][tid], fr[r], a);
    out[(int64_t)u * HD + tid] = __float2bfloat16(a * invL);
  }

  // ---- indicator update (Eq. 2 / Eq. 3) and importance (Eq. 4) of this CTA's slots, its arg-min ----
  if (state_in_smem && rows_alloc > 0 && !mbar_wait(state_bar, 0) && dev_status) atomicExch(dev_status, (int)VATP_ERR_TIMEOUT);
  const bool evicting = hi > B;
  unsigned long long my_key = NO_KEY;
  int my_slot = -1, my_pos = -1;
  {
    // local copies: the stores into the state arrays below cannot alias what the loop reads
    const float* __restrict__ lg = logit_s;
    const float* __restrict__ as = acc_s;
    const float* __restrict__ vs = vn_s;
    const int* __restrict__ ps_s = pos_s;
    float* __restrict__ acc_g = c.acc + (int64_t)u * cap + s0;
#pragma unroll 4
    for (int i = tid; i < cnt; i += WT) {
      const int slot = s0 + i;
      float p;
      if constexpr (GT > 1) {      // the mean of the heads' probabilities
        float a = 0.f;
        for (int h = 0; h < G; ++h) a = fmaf(ex2(lg[h * chunk + i] - gq_mall[h]), gq_invl[h], a);
        p = a / (float)G;
      } else {
        p = ex2(lg[i] - m_all) * invL;
      }
      const bool is_new = slot == fs;
      float S;
      if (WINDOWED) {
        float* ring_row = c.ring + ((int64_t)u * w + (t % w)) * cap;
        const int64_t o = (int64_t)u * cap + slot;
        long long fx;
        if (is_new) {
          fx = prob_to_fixed(p);     // (the recycled slot's ring column is cleared below)
        } else {
          fx = c.acc_fixed[o] + prob_to_fixed(p) - prob_to_fixed(ring_row[slot]);
        }
        ring_row[slot] = p;
        c.acc_fixed[o] = fx;
        S = fixed_to_prob(fx);
      } else {
        S = is_new ? p : (state_in_smem ? as[i] : acc_g[i]) + p;
      }
      if (VATP_INB((int64_t)u * cap + slot, (int64_t)gridDim.x / split * cap, dev_status)) acc_g[i] = S;
      if (evicting) {
        const int ps = is_new ? t : (state_in_smem ? ps_s[i] : c.pos[(int64_t)u * cap + slot]);
        const float I = S * (is_new ? new_norm : (state_in_smem ? vs[i] : c.vnorm[(int64_t)u * cap + slot]));
        if (ps >= F && ps <= t - R) {
          const unsigned long long key = evict_key(I, ps);
          if (key < my_key) { my_key = key; my_slot = slot; my_pos = ps; }
        }
      }
    }
  }
  if (WINDOWED) {
    // recycled slot: the other rows of its ring column belong to the previous occupant (shared out over the unit's CTAs)
    for (int rr = rank * WT + tid; rr < w; rr += split * WT)
      if (rr != t % w && VATP_INB(((int64_t)u * w + rr) * cap + fs, (int64_t)gridDim.x / split * w * cap, dev_status))
        c.ring[((int64_t)u * w + rr) * cap + fs] = 0.f;
  }
  if (!evicting) {
    if (rank == 0 && tid == 0) {
      c.len[u] = hi;
      c.free_slot[u] = hi;
      c.next_pos[u] = t + 1;
      c.last_slot[u] = fs;
      if (evicted) evicted[u] = -1;
    }
    return;
  }
  // this CTA's candidate (positions are unique: exactly one thread holds the winning key), pushed to rank 0
  {
    const unsigned long long wkey = warp_min_key(my_key);
    if (lane == 0) warp_key[wid] = wkey;
    workers_sync<WT>();
    const unsigned long long win = warp_min_key(lane < MW ? warp_key[lane] : NO_KEY);
    Exch* e0 = split > 1 ? cluster.map_shared_rank(&ex, 0) : &ex;
    if (win == NO_KEY) {
      if (tid == 0) e0->key[rank] = NO_KEY;
    } else if (my_key == win) {
      e0->key[rank] = win;
      e0->key_slot[rank] = my_slot;
      e0->key_pos[rank] = my_pos;
    }
  }
  if (split > 1) { cluster_arrive_release(); cluster_wait_acquire(); } else workers_sync<WT>();
  if (rank != 0 || tid != 0) return;      // nothing of the other CTAs' shared memory is read by anyone
  {
    unsigned long long best = NO_KEY;
    int br = -1;
    for (int r = 0; r < split; ++r)
      if (ex.key[r] < best) { best = ex.key[r]; br = r; }
    if (br >= 0) {
      const int slot = ex.key_slot[br];
      if (VATP_INB(slot, cap, dev_status)) c.pos[(int64_t)u * cap + slot] = -1;
      c.free_slot[u] = slot;
      c.len[u] = hi - 1;
      if (evicted) evicted[u] = ex.key_pos[br];
    } else {   // nothing eligible (cannot happen when F + R <= B): keep the state consistent
      c.len[u] = hi;
      c.free_slot[u] = min(hi, cap - 1);
      if (evicted) evicted[u] = -1;
    }
    c.next_pos[u] = t + 1;
    c.last_slot[u] = fs;
  }
}


// Host-side record, per stream, of the buffers the last launches write and of the share of the
// machine each occupies.  Every CTA of a launch stays resident until the previous launch has
// completed, so launch M - j can still be running when M starts only if the launches between them fit
// on the machine together: M may skip all waiting when it touches nothing that those launches write.
struct Range {
  const char* p;
  size_t n;
};
constexpr int HIST = 8, NRANGE = 13;
struct LaunchRecord {
  Range w[NRANGE];
  double share;        // CTAs / (resident CTAs the machine holds of this launch's kind)
};
struct StreamHistory {
  cudaStream_t stream;
  unsigned long long capture;   // 0: launches issued for execution; else the id of the stream capture that recorded them
  bool valid;
  int count, head;     // records held, index of the newest
  LaunchRecord rec[HIST];
};
std::mutex g_hist_mutex;
StreamHistory g_hist[8];
int g_hist_next = 0;

inline bool overlaps(const Range& a, const Range& b) {
  return a.p && b.p && a.n && b.n && a.p < b.p + b.n && b.p < a.p + a.n;
}

// Id of the capture `st` is recording into, 0 when it is not capturing.  Launches recorded into a graph
// keep a history of their own: what was issued for execution before the capture says nothing about what
// precedes a node when the graph is replayed, and the recorded launches are not in flight afterwards.
unsigned long long capture_of(cudaStream_t st) {
  cudaStreamCaptureStatus status = cudaStreamCaptureStatusNone;
  unsigned long long id = 0;
  if (cudaStreamGetCaptureInfo(st, &status, &id) != cudaSuccess) { cudaGetLastError(); return 0; }
  return status == cudaStreamCaptureStatusActive ? (id ? id : ~0ull) : 0;
}

StreamHistory* history_of(cudaStream_t st, unsigned long long capture, bool create) {
  for (auto& x : g_hist)
    if (x.valid && x.stream == st && x.capture == capture) return &x;
  if (!create) return nullptr;
  StreamHistory* h = &g_hist[g_hist_next];
  g_hist_next = (g_hist_next + 1) % 8;
  h->stream = st;
  h->capture = capture;
  h->valid = true;
  h->count = 0;
  h->head = -1;
  return h;
}

// True when `touched` overlaps nothing that a launch possibly still in flight on `st` writes; records this
// launch.  may_overlap false (the caller did not opt in): records it and answers false.
bool independent_of_in_flight(cudaStream_t st, unsigned long long capture, bool may_overlap, const Range* touched, int nt,
                               const Range* written, double share_if_indep, double share_if_not) {
  std::lock_guard<std::mutex> lock(g_hist_mutex);
  StreamHistory* h = history_of(st, capture, true);
  // The first recorded launch follows work this table knows nothing about (another kernel, the start of a
  // graph): it waits, and by the time it lets its successor start everything before it has completed.
  bool indep = may_overlap && h->count > 0;
  double between = 0.0;      // machine share of the launches between the candidate and this one
  for (int j = 0; indep && j < h->count && between < 1.0; ++j) {
    const LaunchRecord& r = h->rec[(h->head - j + HIST) % HIST];
    for (int i = 0; i < nt && indep; ++i)
      for (int k = 0; k < NRANGE; ++k)
        if (overlaps(touched[i], r.w[k])) { indep = false; break; }
    between += r.share;
    if (j == HIST - 1 && between < 1.0 && h->count == HIST) indep = false;   // history too short to tell
  }
  h->head = (h->head + 1) % HIST;
  if (h->count < HIST) ++h->count;
  LaunchRecord& r = h->rec[h->head];
  for (int k = 0; k < NRANGE; ++k) r.w[k] = written[k];
  r.share = indep ? share_if_indep : share_if_not;
  return indep;
}

}  // namespace

// Host-only probe of the overlap policy (no device work): feeds one pretend launch that touches and
// writes the `n` byte ranges [begin[i], begin[i] + bytes[i]) on `stream` and occupies `share` of the
// machine; returns whether it would have been allowed to run beside the launches before it.
bool decode_overlap_policy_probe(void* stream, const uint64_t* begin, const uint64_t* bytes, int n, double share) {
  Range r[NRANGE] = {};
  for (int i = 0; i < n && i < NRANGE; ++i) r[i] = Range{reinterpret_cast<const char*>(begin[i]), (size_t)bytes[i]};
  return independent_of_in_flight(static_cast<cudaStream_t>(stream), 0, true, r, NRANGE, r, share, share);
}

// Any other work this library enqueues on `st` (prefill, selection, compaction, the general decode kernel)
// ends the record: the decode launch after it waits for everything before it.
void decode_history_forget(cudaStream_t st, bool probe_only) {
  const unsigned long long capture = probe_only ? 0 : capture_of(st);
  std::lock_guard<std::mutex> lock(g_hist_mutex);
  if (StreamHistory* h = history_of(st, capture, false)) {
    h->count = 0;
    h->head = -1;
  }
}

// Returns cudaErrorNotSupported when the shape does not fit this kernel's shared memory (the caller
// then takes the general kernel).
cudaError_t launch_decode_mma(const Shape& s, int B, int F, int R, const vatp_cache& c, const void* q, const void* k,
                              const void* v, void* out, int32_t* evicted, int32_t* dev_status, cudaStream_t st,
                              bool may_overlap, int G) {
  const int cap = cache_capacity(B);
  if (!vatp_tc_available() || G < 1 || G > GQ_HEADS) return cudaErrorNotSupported;
  const bool grouped = G > 1;           // s.units counts caches (KV heads); q and out hold G rows per unit
  const int sms = device_sm_count();
  // split a unit over a cluster while the grid still fits on the SMs once (a second launch can then be resident too)
  int split = 1;
  while (split < (grouped ? GQ_MAX_SPLIT : MAX_SPLIT) && s.units * split * 2 <= sms && cap / (split * 2) >= 4 * GROUP) split *= 2;
  int chunk = (cap + split - 1) / split;
  chunk = (chunk + GROUP - 1) / GROUP * GROUP;
  // Shared-memory plan.  A launch that may run beside its neighbours stays within half an SM (two CTAs
  // per SM, so that consecutive launches can both be resident) when at least two stages per warp fit
  // there beside the per-slot state; large caches leave acc / vnorm / pos out of shared memory to get
  // there.  A launch that has to wait for its predecessor anyway runs alone: it takes the whole SM and
  // up to four stages per warp, which doubles the bytes it keeps in flight.
  struct Plan {
    int state_in_smem, nstage;
    size_t dyn;
    bool ok;
  };
  const size_t half_sm = 104 * 1024, whole_sm = 215 * 1024;     // dynamic bytes, 1 KB of it alignment slack
  const size_t tot = (size_t)chunk;      // slots whose logits and state one CTA holds
  auto make_plan = [&](bool alone) {
    Plan p{};
    const int MW = alone ? MW_ALONE : MW_BESIDE;
    const size_t stage_set = (size_t)MW * STAGE_BYTES;
    size_t state_bytes = 4 * sizeof(float) * tot;
    if (grouped)    // logits per head, the state, the streams' partial outputs per head, rank 0's copy of every CTA's
      state_bytes = (size_t)(G + 3) * sizeof(float) * tot + (size_t)(NSTREAM + split) * G * HD * sizeof(float);
    p.state_in_smem = 1;
    const bool fits_half = !alone && state_bytes + 1024 + 2 * stage_set <= half_sm;
    if (!alone && !fits_half && sizeof(float) * tot + 1024 + 2 * stage_set <= half_sm) {
      state_bytes = sizeof(float) * tot;
      p.state_in_smem = tot * 12 <= 2 * stage_set ? 2 : 0;
    }
    p.ok = state_bytes + stage_set + 1024 <= whole_sm;
    if (!p.ok) return p;
    const bool half = !alone && state_bytes + 1024 + 2 * stage_set <= half_sm;
    p.nstage = (int)(((half ? half_sm : whole_sm) - 1024 - state_bytes) / stage_set);
    p.nstage = p.nstage > 4 ? 4 : p.nstage;
    const int groups_per_warp = ((chunk / GROUP) + MW - 1) / MW;
    if (p.nstage > groups_per_warp) p.nstage = groups_per_warp > 0 ? groups_per_warp : 1;
    if (p.state_in_smem == 2 && tot * 12 > (size_t)MW * p.nstage * STAGE_BYTES) p.state_in_smem = 0;
    p.dyn = (size_t)MW * p.nstage * STAGE_BYTES + state_bytes + 1024;
    return p;
  };
  const Plan lone = make_plan(true), beside = grouped ? lone : make_plan(false);      // grouped queries: always a whole SM
  if (!beside.ok || !lone.ok) return cudaErrorNotSupported;
  CUtensorMap tm_k, tm_v;
  if (!make_rows_map_bf16(&tm_k, c.k_cache, (uint64_t)s.units * cap, GROUP) ||
      !make_rows_map_bf16(&tm_v, c.v_cache, (uint64_t)s.units * cap, GROUP))
    return cudaErrorInvalidValue;
  const bool win = s.window > 0;
  const size_t units = (size_t)s.units, slots = units * cap;
  Range written[16] = {{(const char*)c.k_cache, slots * ROW_BYTES}, {(const char*)c.v_cache, slots * ROW_BYTES},
                       {(const char*)c.acc, slots * 4}, {(const char*)c.vnorm, slots * 4}, {(const char*)c.pos, slots * 4},
                       {(const char*)c.len, units * 4}, {(const char*)c.free_slot, units * 4},
                       {(const char*)c.next_pos, units * 4}, {(const char*)c.last_slot, units * 4},
                       {(const char*)out, units * G * ROW_BYTES}, {(const char*)evicted, evicted ? units * 4 : 0},
                       {win ? (const char*)c.ring : nullptr, win ? slots * s.window * 4 : 0},
                       {win ? (const char*)c.acc_fixed : nullptr, win ? slots * 8 : 0},
                       {(const char*)q, units * G * ROW_BYTES}, {(const char*)k, units * ROW_BYTES}, {(const char*)v, units * ROW_BYTES}};
  auto kern_alone = grouped ? (win ? decode_mma_kernel<true, MW_ALONE, GQ_HEADS> : decode_mma_kernel<false, MW_ALONE, GQ_HEADS>)
                            : (win ? decode_mma_kernel<true, MW_ALONE, 1> : decode_mma_kernel<false, MW_ALONE, 1>);
  auto kern_beside = grouped ? kern_alone : (win ? decode_mma_kernel<true, MW_BESIDE, 1> : decode_mma_kernel<false, MW_BESIDE, 1>);
  cudaError_t e = cudaFuncSetAttribute(kern_beside, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)whole_sm);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(kern_alone, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)whole_sm);
  if (e != cudaSuccess) return e;
  // share of the machine this launch holds while resident (every CTA waits for the previous launch before it retires)
  auto share_of = [&](const Plan& p, bool alone) {
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, alone ? kern_alone : kern_beside,
                                                      (alone || grouped ? MW_ALONE : MW_BESIDE) * 32 + 32, p.dyn) != cudaSuccess || occ < 1)
      occ = 1;
    return (double)(s.units * split) / ((double)occ * sms);
  };
  const int independent = independent_of_in_flight(st, capture_of(st), may_overlap, written, 16, written, share_of(beside, false),
                                                   share_of(lone, true)) ? 1 : 0;
  const Plan& pl = independent ? beside : lone;
  auto kern = independent ? kern_beside : kern_alone;
  const int nstage = pl.nstage, state_in_smem = pl.state_in_smem;
  const size_t dyn = pl.dyn;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(s.units * split);
  cfg.blockDim = dim3((independent && !grouped ? MW_BESIDE : MW_ALONE) * 32 + 32);
  cfg.dynamicSmemBytes = dyn;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = split;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start before the previous launch has drained
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kern, tm_k, tm_v, independent, G, state_in_smem, split, chunk, nstage, B, cap, F, R, s.window, s.norm, s.scale * LOG2E, c,
                            (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v,
                            (__nv_bfloat16*)out, evicted, dev_status);
}

}  // namespace vatp
