// Tensor-core prefill scoring for bf16, head_dim 128 (sm_100a: tcgen05 MMA, TMEM accumulators, TMA).
//
// Two launches of one persistent kernel, never materialising the T x T matrix:
//   pass 1  rows = 128 queries (fixed tile), streamed tiles = keys 0..diagonal:
//           per query the running max and sum of exp2 give lse (the normaliser of Eq. 1);
//   pass 2  rows = 128 keys (fixed tile), streamed tiles = queries diagonal..end: S^T = K Q^T is
//           recomputed, every thread owns one key and adds exp2(s - lse_j) over the query columns
//           of its TMEM lane (Eq. 2) - a per-thread running sum, no shuffles, no atomics - then
//           multiplies by the value norm (Eq. 4: l1), which a side warp of pass 1 has reduced.
// Both operands are [token, d] row-major, i.e. K-major for A and B alike.
//
// With a history window (Eq. 3) only the last w query rows count: pass 1 covers the query tiles that
// reach into the window, pass 2 streams from the window's first tile on and also writes the
// probabilities of those rows (win_rows); a side warp zeroes the entries nobody visits.
//
// Warp roles (608 threads): warp 0 TMA producer (it also draws the work items from a global counter,
// works out what they cover and passes that on, and in pass 2 copies the row normalisers of every
// chunk into shared memory beside its tiles), warp 1 MMA issuer and TMEM owner, warps 2-17 four softmax warpgroups (each takes
// one 64-column quarter of every 256-column accumulator, loads it into registers and hands the
// accumulator back at once; four warps per scheduler keep the exponential unit busy where two could
// not), warp 18 the value-norm reduction (pass 1) / window zero fill (pass 2 with Eq. 3).
// Every wait is bounded; on expiry the CTA raises a flag, writes VATP_ERR_TIMEOUT to the status
// word, drains, frees its TMEM and returns.
#include <cuda.h>

#include <mutex>

#include "vatp_internal.cuh"

namespace vatp {
namespace {

constexpr int NSW = 16;            // softmax warps
constexpr int TC_THREADS = (2 + NSW + 1) * 32;
constexpr int TILE = 128;          // rows of the fixed tile = columns of a streamed tile
constexpr int HD = 128;            // head_dim
constexpr int CHUNK = 256;         // streamed tokens per stage = columns of an accumulator
constexpr int NS = 2;              // streamed-chunk stages in shared memory
constexpr int NACC = 2;            // TMEM accumulators (256 columns each)
constexpr int NLSE = 8;            // ring of per-chunk normaliser rows in shared memory (pass 2)
constexpr int SLAB_BYTES = TILE * 128;        // 128 rows x 64 bf16, 128-byte swizzled
constexpr int TILE_BYTES = 2 * SLAB_BYTES;    // two K halves
constexpr int CHUNK_BYTES = 2 * TILE_BYTES;   // 256 rows, two K halves
constexpr uint64_t WAIT_NS = 1000000000ull;
#ifndef VATP_POLY_MASK
#define VATP_POLY_MASK 0x0101   // bit p set: pair p (of the 16 pairs of a 32-column slice) takes the FMA-pipe exponential
#endif

struct Smem {
  alignas(1024) unsigned char fixed[2][TILE_BYTES];      // double-buffered fixed tile
  alignas(1024) unsigned char stream[NS][CHUNK_BYTES];   // [K half][256 rows][128 bytes] per stage
  alignas(128) float nlse[NLSE][CHUNK];  // pass 2: ring of the NEGATED normalisers of the streamed chunks (bulk copies by the producer)
  float part_a[2][3][TILE];   // pass 1: running max of warpgroups 1-3; pass 2: their column sums
  float part_b[2][3][TILE];   // pass 1: running sum of warpgroups 1-3
  alignas(8) uint64_t full[NS], empty[NS];
  uint64_t fixed_full[2], fixed_empty[2];
  uint64_t acc_full[NACC], acc_empty[NACC];
  uint64_t comb_full[2], comb_empty[2];
  uint64_t item_full[4], item_empty[4];   // FIFO of work items from the producer to the other roles
  int item_ring[4][8];                    // u, tile, c_first, c_count, lo (u < 0: no more items)
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(s32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t now_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the CTA is aborting (this or another waiter ran out of time).
// SLEEP_NS > 0 backs off between polls: used by the single-lane producer / MMA roles so that their
// polling does not take issue slots from the softmax warps.
template <int SLEEP_NS = 0>
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* dev_status) {
  if (mbar_try(bar, parity)) return true;
  uint64_t t0 = 0;
  for (uint32_t spins = 1;; ++spins) {
    if (SLEEP_NS > 0) __nanosleep(SLEEP_NS);
    if (mbar_try(bar, parity)) return true;
    if ((spins & 255u) == 0) {
      if (*abort_flag) return false;
      const uint64_t now = now_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > WAIT_NS) {
        *abort_flag = 1;
        if (dev_status) atomicExch(dev_status, (int)VATP_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(s32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(s32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(s32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(s32(bar)), "r"(c0), "r"(c1)
      : "memory");
}

// untiled global -> shared bulk copy; both addresses and the size are multiples of 16 bytes
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(s32(dst)), "l"(src), "r"(bytes), "r"(s32(bar))
               : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M 128, N 128 or 256.
template <int N>
__host__ __device__ constexpr uint32_t idesc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(TILE >> 4) << 24);
}

// One 128 x N x 16 MMA.  ACC = false overwrites the accumulator, true adds to it.  Issued by a
// single thread, so every instruction between two MMAs costs tensor-pipe time: the descriptors are
// built once per tile and advanced by adding compile-time constants.
template <bool ACC, int N>
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc<N>()), "n"(ACC ? 1 : 0)
      : "memory");
}
// Descriptor offsets (16-byte units) of the kk-th 16-element K step.  The fixed tile is two slabs of
// 128 rows; a streamed chunk is two slabs of 256 rows.
__host__ __device__ constexpr uint64_t k_off_fixed(int kk) { return (uint64_t)(((kk / 4) * SLAB_BYTES + (kk % 4) * 32) >> 4); }
__host__ __device__ constexpr uint64_t k_off_stream(int kk) { return (uint64_t)(((kk / 4) * 2 * SLAB_BYTES + (kk % 4) * 32) >> 4); }
template <int KK, int N>
__device__ __forceinline__ void umma_tile(uint32_t d_addr, uint64_t da, uint64_t db) {
  if constexpr (KK < HD / 16) {
    umma_bf16<(KK > 0), N>(d_addr, da + k_off_fixed(KK), db + k_off_stream(KK));
    umma_tile<KK + 1, N>(d_addr, da, db);
  }
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t addr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(addr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Packed fp32 pairs (fma.rn.f32x2 / add.rn.f32x2): one issue slot does two lanes' worth of FMA work.
// The softmax warps are bound by instruction issue, not by the FMA pipe, so packing halves the cost
// of everything around the exponential.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pk2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void upk2(f32x2 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float hsum2(f32x2 v) {
  float a, b;
  upk2(v, a, b);
  return a + b;
}

// exp2 of a pair on the special-function unit (16 results per clock per SM)
__device__ __forceinline__ f32x2 ex2_sfu2(f32x2 v) {
  float a, b;
  upk2(v, a, b);
  return pk2(ex2(a), ex2(b));
}
// exp2 of a pair on the FMA pipe: round-to-nearest split x = n + f with f in [-0.5, 0.5] (adding
// 1.5 * 2^23 leaves n in the low mantissa bits), a degree-3 minimax polynomial for 2^f (relative
// error 7.5e-5) and an exponent-field add for 2^n.  The special-function unit alone would bound the
// kernel below the tensor pipe; a share of the pairs (VATP_POLY_MASK) goes here instead.
__device__ __forceinline__ f32x2 ex2_fma2(f32x2 v) {
  float a, b;
  upk2(v, a, b);
  v = pk2(fmaxf(a, -126.f), fmaxf(b, -126.f));
  const f32x2 t = add2(v, pk2(12582912.f, 12582912.f));
  const f32x2 r = add2(t, pk2(-12582912.f, -12582912.f));
  const f32x2 f = fma2(r, pk2(-1.f, -1.f), v);
  f32x2 p = fma2(pk2(0.05517164617776871f, 0.05517164617776871f), f, pk2(0.2426111251115799f, 0.2426111251115799f));
  p = fma2(p, f, pk2(0.6932609677314758f, 0.6932609677314758f));
  p = fma2(p, f, pk2(0.9999280571937561f, 0.9999280571937561f));
  float tl, th, pl, ph;
  upk2(t, tl, th);
  upk2(p, pl, ph);
  return pk2(__int_as_float(__float_as_int(pl) + (__float_as_int(tl) << 23)),
             __int_as_float(__float_as_int(ph) + (__float_as_int(th) << 23)));
}
// pair index p in 0..15 of a slice: compile-time choice of the pipe
__device__ __forceinline__ f32x2 exp2_pair(int p, f32x2 v) {
  if ((VATP_POLY_MASK >> p) & 1) return ex2_fma2(v);
  return ex2_sfu2(v);
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// pass 1 building blocks for one 32-column slice (x: raw dot products of this thread's query row)
__device__ __forceinline__ void mask_after_diagonal(float (&x)[32], int c0, int row) {
#pragma unroll
  for (int i = 0; i < 32; ++i)
    if (c0 + i > row) x[i] = -INFINITY;
}
__device__ __forceinline__ float slice_max(const float (&x)[32]) {
  // four short max chains instead of one long one
  float c0m = max3(x[0], x[1], x[2]), c1m = max3(x[8], x[9], x[10]);
  float c2m = max3(x[16], x[17], x[18]), c3m = max3(x[24], x[25], x[26]);
  c0m = max3(c0m, x[3], x[4]); c1m = max3(c1m, x[11], x[12]); c2m = max3(c2m, x[19], x[20]); c3m = max3(c3m, x[27], x[28]);
  c0m = max3(c0m, x[5], x[6]); c1m = max3(c1m, x[13], x[14]); c2m = max3(c2m, x[21], x[22]); c3m = max3(c3m, x[29], x[30]);
  c0m = max3(c0m, x[7], c1m); c2m = max3(c2m, x[15], c3m);
  return max3(c0m, c2m, fmaxf(x[23], x[31]));
}
// sum over the slice of exp2(scale_log2 * x - m)
__device__ __forceinline__ float slice_exp_sum(const float (&x)[32], float scale_log2, float m) {
  const f32x2 c2 = pk2(scale_log2, scale_log2), nm2 = pk2(-m, -m);
  f32x2 a0 = pk2(0.f, 0.f), a1 = a0;
#pragma unroll
  for (int i = 0; i < 32; i += 4) {
    a0 = add2(a0, exp2_pair(i >> 1, fma2(pk2(x[i], x[i + 1]), c2, nm2)));
    a1 = add2(a1, exp2_pair((i >> 1) + 1, fma2(pk2(x[i + 2], x[i + 3]), c2, nm2)));
  }
  return hsum2(add2(a0, a1));
}

// One 32-column slice of an accumulator row.  x holds raw dot products; c0 is the slice's first
// column inside the tile, row the thread's row.
//   PASS 1 (row = query, columns = keys): online max / sum of exp2(scale_log2 * s); on the diagonal
//           tile keys beyond the query are masked.
//   PASS 2 (row = key, columns = queries): cs += exp2(scale_log2 * s - lse2[query]); on the diagonal
//           tile queries before the key are masked.  nlse_t: the tile's 128 NEGATED normalisers in
//           shared memory.  cs: two packed pairs of running sums.
//   WIN (pass 2, Eq. 3): the probabilities themselves are also written out, column i of the slice to
//           wo.p[i * wo.T] for wo.lo <= i < wo.hi (the rows of the last-w-queries window).
struct WinOut {
  float* p;
  int lo, hi;
  int64_t T;
  char* base;      // all 32 columns live (lo == 0, hi == 32): this unit's window block (same for the whole warp) ...
  uint32_t off;    // ... and this thread's byte offset of column 0 in it; columns are row4 bytes apart
  uint32_t row4;
  bool full;
};
// Four consecutive window rows of one key.  The common case (whole slice inside the window and the prompt) is one
// 32-bit multiply-add and one store per value on a warp-uniform base; ragged slices test every column.
__device__ __forceinline__ void win_store4(const WinOut& wo, int i, float p0, float p1, float p2, float p3) {
  if (wo.full) {
    *reinterpret_cast<float*>(wo.base + (wo.off + (uint32_t)i * wo.row4)) = p0;
    *reinterpret_cast<float*>(wo.base + (wo.off + (uint32_t)(i + 1) * wo.row4)) = p1;
    *reinterpret_cast<float*>(wo.base + (wo.off + (uint32_t)(i + 2) * wo.row4)) = p2;
    *reinterpret_cast<float*>(wo.base + (wo.off + (uint32_t)(i + 3) * wo.row4)) = p3;
  } else {
    if (i >= wo.lo && i < wo.hi) wo.p[i * wo.T] = p0;
    if (i + 1 >= wo.lo && i + 1 < wo.hi) wo.p[(i + 1) * wo.T] = p1;
    if (i + 2 >= wo.lo && i + 2 < wo.hi) wo.p[(i + 2) * wo.T] = p2;
    if (i + 3 >= wo.lo && i + 3 < wo.hi) wo.p[(i + 3) * wo.T] = p3;
  }
}
template <int PASS, bool DIAG, bool WIN>
__device__ __forceinline__ void consume32(float (&x)[32], int c0, int row, float scale_log2, float& m_run, float& l_run,
                                          f32x2 (&cs)[2], const float* nlse_t, const WinOut& wo) {
  const f32x2 c2 = pk2(scale_log2, scale_log2);
  if (PASS == 1) {
    if (DIAG) mask_after_diagonal(x, c0, row);
    const float cmax = slice_max(x) * scale_log2;   // scale > 0 keeps the order
    const float m_new = fmaxf(m_run, cmax);
    l_run *= ex2(fmaxf(m_run - m_new, -126.f));      // (-inf) - (-inf) = NaN -> -126 -> factor on a zero sum
    m_run = m_new;
    l_run += slice_exp_sum(x, scale_log2, m_run);
  } else if (!DIAG) {
    // explicit shared-memory loads: through the generic pointer they would take the slower generic path
    const uint32_t lp = s32(nlse_t + c0);
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
      ulonglong2 L;
      asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(L.x), "=l"(L.y) : "r"(lp + 4 * i));
      const f32x2 e0 = exp2_pair(i >> 1, fma2(pk2(x[i], x[i + 1]), c2, L.x));
      const f32x2 e1 = exp2_pair((i >> 1) + 1, fma2(pk2(x[i + 2], x[i + 3]), c2, L.y));
      cs[0] = add2(cs[0], e0);
      cs[1] = add2(cs[1], e1);
      if (WIN) {
        float p0, p1, p2, p3;
        upk2(e0, p0, p1);
        upk2(e1, p2, p3);
        win_store4(wo, i, p0, p1, p2, p3);
      }
    }
  } else {
    const uint32_t lp = s32(nlse_t + c0);
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
      float4 L;
      asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(L.x), "=f"(L.y), "=f"(L.z), "=f"(L.w) : "r"(lp + 4 * i));
      float p0 = ex2(fmaf(x[i], scale_log2, L.x));
      float p1 = ex2(fmaf(x[i + 1], scale_log2, L.y));
      float p2 = ex2(fmaf(x[i + 2], scale_log2, L.z));
      float p3 = ex2(fmaf(x[i + 3], scale_log2, L.w));
      if (c0 + i < row) p0 = 0.f;
      if (c0 + i + 1 < row) p1 = 0.f;
      if (c0 + i + 2 < row) p2 = 0.f;
      if (c0 + i + 3 < row) p3 = 0.f;
      s0 += p0; s1 += p1; s2 += p2; s3 += p3;
      if (WIN) {
        win_store4(wo, i, p0, p1, p2, p3);
      }
    }
    cs[0] = add2(cs[0], pk2(s0, s1));
    cs[1] = add2(cs[1], pk2(s2, s3));
  }
}

struct TcArgs {
  int units, heads, T, nt, nch, Tpad;  // nt tiles of 128 tokens, nch = ceil(nt / 2) chunks, Tpad = 256 nch
  // Grouped queries in one launch (G > 1): the units are the query heads, unit (b, h) reads K and V of KV head h / G;
  // value norms exist per KV unit, and pass 2 writes query head h's indicator to slice h % G of attn_acc
  // ([G][kv_units][T]: the group mean is taken afterwards) and no score.  G = 1: kv_units = units, kv_heads = heads.
  int G, kv_units, kv_heads;
  float scale_log2;
  const __nv_bfloat16* v;
  int64_t sb, sh, st;       // element strides of v
  float* lse2;              // [units][Tpad] NEGATED log2-domain row normalisers (-inf where no query counts)
  float* lse_out;           // natural-log copy, nullable: unit (b, h)'s T values start at b * lse_sb + h * lse_sh
  int64_t lse_sb, lse_sh;
  int64_t out_sb, out_sh;   // fused forward: unit (b, h)'s output rows start at b * out_sb + h * out_sh (elements)
  float* attn_acc;
  float* vnorm;
  float* score;
  int32_t* dev_status;
  // Eq. 3 (last w queries): only query rows >= first_row count; ft = first_row / 128; win_rows row r is
  // query wrow0 + r (wrow0 = T - w, negative when the prompt is shorter than the window).  H2O: all zero.
  int first_row, ft, wrow0, window;
  int gu;                   // units per scheduling group (their K and Q fit in L2 together)
  int norm;                 // vatp_norm_kind of the value norm
  int side_norm;            // pass 1 reduces the value norms in its side warp (else vnorm_kernel has, before it)
  unsigned* counters;       // [2] next work item of pass 1 / pass 2 (zeroed before pass 1 is launched)
  int wait_first;           // pass 1 was launched as a programmatic dependent (of the kernel that zeroes the counters):
                            // nothing in global memory is touched before griddepcontrol.wait
  float* win_rows;
};

// Work items are (unit, fixed tile of 128 rows), longest first within a group of units whose K and Q
// share the L2 (with hundreds of units the streamed operand would otherwise come from HBM every
// time).  The persistent CTAs draw them from a global counter, so a CTA that finishes early takes
// the next item instead of idling (a static deal left the average CTA idle for a tenth of a pass).  The other operand
// streams in chunks of 256 tokens (two tiles), so that one MMA instruction is 128 x 256 x 16: a
// single thread issues the MMAs, and at 128 x 128 x 16 the issue cost exceeds the execution time.
//   PASS 1: fixed = query tile i, streamed key chunks 0 .. i/2       (key tile kt needed iff kt <= i);
//           with a history window only the query tiles that reach into it are items
//   PASS 2: fixed = key tile i, streamed query chunks lo/2 .. nch-1  (query tile qt needed iff lo <= qt < nt,
//           lo = max(i, first tile of the window))
// Softmax warpgroup g takes columns [128 g, 128 g + 128) of every accumulator, i.e. streamed tile
// 2 c + g of chunk c; the two partial results of a row are combined once per item.

struct Item {
  int u, tile, c_first, c_count;
  int lo;   // pass 2: first query tile that counts for this key tile
};
// the KV unit whose keys and values unit u attends over
__device__ __forceinline__ int kv_unit_of(const TcArgs& a, int u) {
  if (a.G == 1) return u;
  const int b = u / a.heads, h = u - b * a.heads;
  return b * a.kv_heads + h / a.G;
}
template <int PASS>
__device__ __forceinline__ Item item_of(int id, const TcArgs& a) {
  Item it;
  // units are taken in groups whose K and Q stay in L2 together; inside a group, longest items first
  const int ntp = PASS == 1 ? a.nt - a.ft : a.nt;
  const int grp = id / (a.gu * ntp);
  const int rem = id - grp * (a.gu * ntp);
  const int u0 = grp * a.gu;
  const int nu = min(a.gu, a.units - u0);
  const int r = rem / nu;
  it.u = u0 + (rem - r * nu);
  if (PASS == 1) { it.tile = a.nt - 1 - r; it.c_first = 0; it.c_count = it.tile / 2 + 1; it.lo = 0; }
  else           { it.tile = r; it.lo = max(r, a.ft); it.c_first = it.lo / 2; it.c_count = a.nch - it.c_first; }
  return it;
}
// is streamed tile st (= 2 * chunk + half) needed by the item?
template <int PASS>
__device__ __forceinline__ bool tile_needed(const Item& it, int st, int nt) {
  return PASS == 1 ? st <= it.tile : (st >= it.lo && st < nt);
}

// Value norms of all (unit, token tile) pairs, shared out over the CTAs: the work of pass 1's side warp.
template <int KIND>
__device__ __forceinline__ void side_value_norms(const TcArgs& a, int lane) {
  for (int id = blockIdx.x; id < a.kv_units * a.nt; id += gridDim.x) {
    Item it;
    it.tile = id / a.kv_units;
    it.u = id - it.tile * a.kv_units;      // a KV unit
    const int b = it.u / a.kv_heads, h = it.u - b * a.kv_heads;
    const __nv_bfloat16* vu = a.v + (int64_t)b * a.sb + (int64_t)h * a.sh;
    // 16 lanes per row, two rows per load instruction, 16 rows in flight per lane group
    const int sub = lane >> 4, part = lane & 15;
    for (int r0 = 0; r0 < TILE; r0 += 32) {
      uint4 raw[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int tok = it.tile * TILE + r0 + 2 * j + sub;
        raw[j] = make_uint4(0u, 0u, 0u, 0u);
        if (tok < a.T) raw[j] = __ldg(reinterpret_cast<const uint4*>(vu + (int64_t)tok * a.st) + part);
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const uint32_t w[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
        float acc = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i)
          acc = norm_fold(KIND, norm_fold(KIND, acc, __uint_as_float(w[i] << 16)), __uint_as_float(w[i] & 0xffff0000u));
#pragma unroll
        for (int o = 8; o; o >>= 1) acc = norm_merge(KIND, acc, __shfl_xor_sync(0xffffffffu, acc, o));
        const int tok = it.tile * TILE + r0 + 2 * j + sub;
        if (part == 0 && tok < a.T && VATP_INB((int64_t)it.u * a.T + tok, (int64_t)a.kv_units * a.T, a.dev_status))
          a.vnorm[(int64_t)it.u * a.T + tok] = norm_finish(KIND, acc);
      }
    }
  }
}

template <int PASS, bool WIN>
__global__ void __launch_bounds__(TC_THREADS, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k, TcArgs a) {
  extern __shared__ unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  volatile int* abort_flag = &sm.abort_flag;
  const int items = a.units * (PASS == 1 ? a.nt - a.ft : a.nt);

  if (tid == 0) {
    for (int i = 0; i < NS; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sm.fixed_full[i], 1); mbar_init(&sm.fixed_empty[i], 1);
      mbar_init(&sm.comb_full[i], 3 * 128); mbar_init(&sm.comb_empty[i], 128);
    }
    for (int i = 0; i < NACC; ++i) { mbar_init(&sm.acc_full[i], 1); mbar_init(&sm.acc_empty[i], NSW); }
    // consumers of the item FIFO: the MMA warp, eight softmax warps and, for Eq. 3's pass 2, the side warp
    for (int i = 0; i < 4; ++i) { mbar_init(&sm.item_full[i], 1); mbar_init(&sm.item_empty[i], 1 + NSW + ((PASS == 2 && WIN) ? 1 : 0)); }
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (wid == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(&sm.tmem_base)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  if (PASS == 1 && a.wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");

  // Consumer side of the item FIFO: the itl-th item of this CTA (u < 0 ends the pass, also when the CTA
  // is aborting).  The producer has worked out what the item covers, once for the whole CTA (the index
  // arithmetic takes several integer divisions).  The slot is handed back as soon as it has been read.
  auto next_item = [&](uint32_t itl, bool whole_warp) -> Item {
    const int slot = itl & 3;
    bool got = mbar_wait(&sm.item_full[slot], (itl >> 2) & 1, abort_flag, a.dev_status);
    if (whole_warp) got = __all_sync(0xffffffffu, got);
    Item it{-1, 0, 0, 0, 0};
    if (got) {
      const volatile int* f = &sm.item_ring[slot][0];
      it.u = f[0]; it.tile = f[1]; it.c_first = f[2]; it.c_count = f[3]; it.lo = f[4];
    }
    if (whole_warp) __syncwarp();
    if (got && (!whole_warp || lane == 0)) mbar_arrive(&sm.item_empty[slot]);
    return it;
  };

  // the operand that stays fixed per item and the one that streams
  const CUtensorMap* tm_fixed = PASS == 1 ? &tm_q : &tm_k;
  const CUtensorMap* tm_stream = PASS == 1 ? &tm_k : &tm_q;

  // Pass 2 is launched as a programmatic dependent of pass 1: its CTAs start as pass-1 CTAs retire and
  // set up, fetch items and stream Q / K tiles at once; only what pass 1 writes (normalisers, value
  // norms) is read after griddepcontrol.wait, i.e. once pass 1 has completed.
  // (Pass 2 in turn releases whatever follows it; vatp_select, launched the same way, reads the scores
  // only after its own griddepcontrol.wait.)
  if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (wid == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      bool waited_for_pass1 = false;
      uint32_t n = 0;
      int next = (int)atomicAdd(&a.counters[PASS - 1], 1u);
      for (uint32_t itl = 0; ok; ++itl) {
        const int id = next;
        const int slot = itl & 3;
        Item it{-1, 0, 0, 0, 0};
        if (id < items) it = item_of<PASS>(id, a);
        ok = mbar_wait<20>(&sm.item_empty[slot], ((itl >> 2) & 1) ^ 1, abort_flag, a.dev_status);
        if (!ok) break;
        {
          volatile int* f = &sm.item_ring[slot][0];
          f[0] = it.u; f[1] = it.tile; f[2] = it.c_first; f[3] = it.c_count; f[4] = it.lo;
        }
        mbar_arrive(&sm.item_full[slot]);
        if (id >= items) break;
        next = (int)atomicAdd(&a.counters[PASS - 1], 1u);     // in flight while this item's tiles are requested
        const int b = it.u / a.heads, h = it.u - b * a.heads;
        const int fb = itl & 1;
        // head coordinate of the fixed and of the streamed operand (K is the streamed one in pass 1, the fixed one in pass 2)
        const int hk = a.G > 1 ? h / a.G : h;
        const int h_fix = PASS == 1 ? h : hk, h_str = PASS == 1 ? hk : h;
        ok = mbar_wait<20>(&sm.fixed_empty[fb], ((itl >> 1) & 1) ^ 1, abort_flag, a.dev_status);
        if (!ok) break;
        mbar_expect_tx(&sm.fixed_full[fb], TILE_BYTES);
        tma_load_4d(sm.fixed[fb], tm_fixed, &sm.fixed_full[fb], 0, it.tile * TILE, h_fix, b);
        tma_load_4d(sm.fixed[fb] + SLAB_BYTES, tm_fixed, &sm.fixed_full[fb], 64, it.tile * TILE, h_fix, b);
        for (int c = 0; c < it.c_count; ++c, ++n) {
          const int stg = n % NS;
          ok = mbar_wait<20>(&sm.empty[stg], ((n / NS) & 1) ^ 1, abort_flag, a.dev_status);
          if (!ok) break;
          // chunk layout: [K half][256 rows][128 bytes]; rows beyond T arrive as zeros
          const int tok0 = (it.c_first + c) * CHUNK;
          mbar_expect_tx(&sm.full[stg], CHUNK_BYTES + (PASS == 2 ? CHUNK * 4 : 0));
#pragma unroll
          for (int kh = 0; kh < 2; ++kh)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh)
              tma_load_4d(sm.stream[stg] + kh * (2 * SLAB_BYTES) + hh * SLAB_BYTES, tm_stream, &sm.full[stg], 64 * kh,
                          tok0 + hh * TILE, h_str, b);
          if (PASS == 2) {
            // The chunk's 256 normalisers travel with its tiles and are complete when its MMAs are.  Ring slot
            // n % NLSE: the MMAs of chunk n - 2 have completed (that freed this stage), so every softmax warp
            // has handed back accumulator n - 4 and is past the normalisers of chunk n - 5 and of all before it.
            // They are pass 1's output: nothing of it is read before that launch has completed.
            if (!waited_for_pass1) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited_for_pass1 = true; }
            if (VATP_INB((int64_t)it.u * a.Tpad + tok0 + CHUNK - 1, (int64_t)a.units * a.Tpad, a.dev_status))
              bulk_load(sm.nlse[n % NLSE], a.lse2 + (int64_t)it.u * a.Tpad + tok0, CHUNK * 4, &sm.full[stg]);
          }
        }
      }
    }
  } else if (wid == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      uint32_t n = 0;
      const uint64_t stage_desc0 = umma_desc(s32(sm.stream[0]));   // stages are CHUNK_BYTES apart
      const uint64_t fixed_desc0 = umma_desc(s32(sm.fixed[0]));    // buffers are TILE_BYTES apart
      for (uint32_t itl = 0; ok; ++itl) {
        const Item it = next_item(itl, false);
        if (it.u < 0) break;
        if (!VATP_INB(it.u, a.units, a.dev_status) || !VATP_INB(it.tile, a.nt, a.dev_status) ||
            !VATP_INB(it.c_first + it.c_count - 1, a.nch, a.dev_status)) break;
        const int fb = itl & 1;
        ok = mbar_wait(&sm.fixed_full[fb], (itl >> 1) & 1, abort_flag, a.dev_status);
        if (!ok) break;
        const uint64_t fixed_desc = fixed_desc0 + (uint64_t)fb * (TILE_BYTES >> 4);
        for (int c = 0; c < it.c_count; ++c, ++n) {
          const int stg = n % NS, ab = n % NACC;
          ok = mbar_wait(&sm.full[stg], (n / NS) & 1, abort_flag, a.dev_status) &&
               mbar_wait(&sm.acc_empty[ab], ((n / NACC) & 1) ^ 1, abort_flag, a.dev_status);
          if (!ok) break;
          tc_fence_after();
          const int st0 = 2 * (it.c_first + c);
          const bool need0 = tile_needed<PASS>(it, st0, a.nt), need1 = tile_needed<PASS>(it, st0 + 1, a.nt);
          const uint64_t stream_desc = stage_desc0 + (uint64_t)stg * (CHUNK_BYTES >> 4);
          const uint32_t d_addr = tmem + ab * CHUNK;
          if (need0 && need1)      umma_tile<0, 256>(d_addr, fixed_desc, stream_desc);
          else if (need0)          umma_tile<0, 128>(d_addr, fixed_desc, stream_desc);
          else                     umma_tile<0, 128>(d_addr + TILE, fixed_desc, stream_desc + (SLAB_BYTES >> 4));
          umma_commit(&sm.empty[stg]);      // the chunk may be overwritten once these MMAs have read it
          umma_commit(&sm.acc_full[ab]);    // accumulator ready for the softmax warps
        }
        if (ok) umma_commit(&sm.fixed_empty[fb]);
      }
    }
  } else if (wid < 2 + NSW) {
    // ------------------------------------------------------------------ softmax warpgroups
    const int sw = wid - 2;
    const int g = sw >> 2;                        // warpgroup g takes columns [64 g, 64 g + 64) of every accumulator
    const int quarter = wid & 3;                  // TMEM lanes this warp may touch
    const int row = quarter * 32 + lane;          // row of the fixed tile = TMEM lane
    const int half = g >> 1;                      // which 128-token tile of a chunk those columns belong to
    const int cbase = (g & 1) * 64;               // and where they start inside that tile
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16) + half * TILE + cbase;
    bool ok = true;
    uint32_t n = 0;
    if (PASS == 2) asm volatile("griddepcontrol.wait;" ::: "memory");
    for (uint32_t itl = 0; ok; ++itl) {
      const Item it = next_item(itl, true);
      if (it.u < 0) break;
      const int u = it.u;
      const int pi = itl & 1;
      const uint32_t ipar = (itl >> 1) & 1;
      const int tok = it.tile * TILE + row;       // query (pass 1) or key (pass 2) index of this thread
      // pass 2: this key's value norm, written by pass 1; fetched now, used in the item's epilogue
      float n1 = 0.f;
      if (PASS == 2 && g == 0 && tok < a.T) n1 = __ldg(a.vnorm + (int64_t)kv_unit_of(a, u) * a.T + tok);
      float m_run = -INFINITY, l_run = 0.f;       // pass 1
      f32x2 cs[2] = {pk2(0.f, 0.f), pk2(0.f, 0.f)};   // pass 2: four running sums, packed
      const uint32_t n0 = n;
      n += it.c_count;
      // streamed tile this warp's columns belong to in chunk c, and whether the item needs it
      auto st_of = [&](int c) { return 2 * (it.c_first + c) + half; };
      auto needed = [&](int c) { return tile_needed<PASS>(it, st_of(c), a.nt); };
      // where the probabilities of the 32 query columns starting at column c0 of streamed tile stile go (Eq. 3 rows)
      auto wout = [&](int stile, int c0) {
        WinOut wo{nullptr, 0, 0, 0, nullptr, 0u, 0u, false};
        if (WIN && PASS == 2) {
          const int q0 = stile * TILE + c0;
          wo.T = a.T;
          wo.lo = min(max(a.first_row - q0, 0), 32);
          wo.hi = tok < a.T ? min(max(a.T - q0, 0), 32) : 0;
          wo.p = a.win_rows + ((int64_t)u * a.window + (q0 - a.wrow0)) * a.T + tok;
          // a unit's window block is window * T * 4 bytes: 32-bit offsets while that stays below 4 GB
          wo.full = wo.lo == 0 && wo.hi == 32 && (uint64_t)a.window * a.T < (1ull << 30);
          wo.base = reinterpret_cast<char*>(a.win_rows + (int64_t)u * a.window * a.T);
          wo.off = wo.full ? ((uint32_t)(q0 - a.wrow0) * (uint32_t)a.T + (uint32_t)tok) * 4u : 0u;
          wo.row4 = (uint32_t)a.T * 4u;
#ifdef VATP_DEBUG_BOUNDS
          // the first and the last window entry this slice may write
          const int64_t lim = (int64_t)a.units * a.window * a.T;
          if (wo.hi > wo.lo && (!VATP_INB((wo.p - a.win_rows) + (int64_t)wo.lo * a.T, lim, a.dev_status) ||
                                !VATP_INB((wo.p - a.win_rows) + (int64_t)(wo.hi - 1) * a.T, lim, a.dev_status))) {
            wo.lo = wo.hi = 0;
            wo.full = false;
          }
#endif
        }
        return wo;
      };
      for (int c = 0; c < it.c_count; ++c) {
        const uint32_t ab = (n0 + c) % NACC;
        bool w = mbar_wait(&sm.acc_full[ab], ((n0 + c) / NACC) & 1, abort_flag, a.dev_status);
        w = __all_sync(0xffffffffu, w);
        if (!w) { ok = false; break; }
        tc_fence_after();
        if (!needed(c)) {
          // this tile of the chunk is masked for the item: hand the accumulator back at once
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.acc_empty[ab]);
          continue;
        }
        // The warp's 64 columns are taken as two waves of 32: with one wave of accumulator values live
        // the compiler has registers left to keep several exponentials in flight.
        float x[32];
        const uint32_t t_addr = lane_addr + ab * CHUNK;
        const int stile = st_of(c);
        // pass 2: the chunk's negated normalisers arrived with its tiles (the accumulator being complete
        // implies that those copies are); indexed by the column inside this warp's tile
        const float* lse_t = sm.nlse[(n0 + c) % NLSE] + half * TILE;
        if (!VATP_INB(it.u, a.units, a.dev_status) || !VATP_INB(tok - row, (int64_t)a.nt * TILE, a.dev_status)) { ok = false; break; }
        tmem_ld32(t_addr, x);
        tmem_ld_wait();
        if (stile == it.tile) consume32<PASS, true, WIN>(x, cbase, row, a.scale_log2, m_run, l_run, cs, lse_t, wout(stile, cbase));
        else                  consume32<PASS, false, WIN>(x, cbase, row, a.scale_log2, m_run, l_run, cs, lse_t, wout(stile, cbase));
        tmem_ld32(t_addr + 32, x);
        tmem_ld_wait();
        // all of this warp's columns have been read: the MMA warp may overwrite them
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.acc_empty[ab]);
        if (stile == it.tile) consume32<PASS, true, WIN>(x, cbase + 32, row, a.scale_log2, m_run, l_run, cs, lse_t, wout(stile, cbase + 32));
        else                  consume32<PASS, false, WIN>(x, cbase + 32, row, a.scale_log2, m_run, l_run, cs, lse_t, wout(stile, cbase + 32));
      }
      if (!ok) break;
      // ---- end of item: warpgroups 1-3 hand their partials to warpgroup 0, which finishes the rows
      if (g > 0) {
        ok = mbar_wait(&sm.comb_empty[pi], ipar ^ 1, abort_flag, a.dev_status);
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
        if (PASS == 1) { sm.part_a[pi][g - 1][row] = m_run; sm.part_b[pi][g - 1][row] = l_run; }
        else           { sm.part_a[pi][g - 1][row] = hsum2(add2(cs[0], cs[1])); }
        mbar_arrive(&sm.comb_full[pi]);
      } else {
        ok = mbar_wait(&sm.comb_full[pi], ipar, abort_flag, a.dev_status);
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
        if (PASS == 1) {
          const float m1 = sm.part_a[pi][0][row], m2 = sm.part_a[pi][1][row], m3 = sm.part_a[pi][2][row];
          const float l1 = sm.part_b[pi][0][row], l2 = sm.part_b[pi][1][row], l3 = sm.part_b[pi][2][row];
          mbar_arrive(&sm.comb_empty[pi]);
          const float m = fmaxf(fmaxf(m_run, m1), fmaxf(m2, m3));
          float l = 0.f;
          if (l_run > 0.f) l += l_run * ex2(m_run - m);
          if (l1 > 0.f) l += l1 * ex2(m1 - m);
          if (l2 > 0.f) l += l2 * ex2(m2 - m);
          if (l3 > 0.f) l += l3 * ex2(m3 - m);
          const float lse2 = m + log2f(l);
          // queries outside the prompt or before the history window contribute nothing to pass 2
          // (stored negated: pass 2 adds it to the scaled dot product)
          if (VATP_INB((int64_t)u * a.Tpad + tok, (int64_t)a.units * a.Tpad, a.dev_status))
            a.lse2[(int64_t)u * a.Tpad + tok] = (tok < a.T && tok >= a.first_row) ? -lse2 : -INFINITY;
          // an odd tile count leaves half a chunk of padding that pass 2 reads as "no query"
          if ((a.nt & 1) && it.tile == a.nt - 1 && VATP_INB((int64_t)u * a.Tpad + tok + TILE, (int64_t)a.units * a.Tpad, a.dev_status))
            a.lse2[(int64_t)u * a.Tpad + tok + TILE] = -INFINITY;
          if (a.lse_out && tok < a.T)
            a.lse_out[(int64_t)(u / a.heads) * a.lse_sb + (int64_t)(u % a.heads) * a.lse_sh + tok] = lse2 * 0.69314718055994531f;
        } else {
          const float tot = hsum2(add2(cs[0], cs[1])) + (sm.part_a[pi][0][row] + sm.part_a[pi][1][row]) + sm.part_a[pi][2][row];
          mbar_arrive(&sm.comb_empty[pi]);
          if (tok < a.T && VATP_INB((int64_t)u * a.T + tok, (int64_t)a.units * a.T, a.dev_status)) {
            if (a.G == 1) {
              const int64_t o = (int64_t)u * a.T + tok;
              a.attn_acc[o] = tot;
              a.score[o] = tot * n1;
            } else {      // query head h's indicator: slice h % G of the partial indicators, row of its KV unit
              const int h = u % a.heads;
              a.attn_acc[((int64_t)(h % a.G) * a.kv_units + kv_unit_of(a, u)) * a.T + tok] = tot;
            }
          }
        }
      }
    }
  } else if (PASS == 1 && a.side_norm) {
    // ------------------------------------------------------------------ value norms (Eq. 4), the side warp
    // Independent of the attention work of this pass: the CTAs share out all (unit, token tile) pairs,
    // so these warps cover every token.  Pass 2 reads the norms back in its epilogue.
    // Only Eq. 4's own l1 norm is taken here.  This warp shares a scheduler with four softmax warps and
    // gets few issue slots: with the square and root of the l2 variant it became the last thing to
    // finish in every CTA and the whole pass a fifth longer, so the ablation's variants go to the
    // kernel below instead.
    side_value_norms<VATP_NORM_L1>(a, lane);
  } else if (WIN) {
    // ------------------------------------------------------------------ pass 2, Eq. 3: window rows nobody visits
    // For key tile i the query tiles before it are never streamed (causal), and when the prompt is
    // shorter than the window its first rows belong to no query: those entries of win_rows are zero.
    for (uint32_t itl = 0;; ++itl) {
      const Item it = next_item(itl, true);
      if (it.u < 0) break;
      float* wr = a.win_rows + (int64_t)it.u * a.window * a.T;
      const int k0 = it.tile * TILE;
      const int r_end = min(it.tile * TILE, a.T) - a.wrow0;      // rows of queries before this key tile
      for (int r = 0; r < min(r_end, a.window); ++r)
        for (int kk = lane; kk < TILE; kk += 32)
          if (k0 + kk < a.T) wr[(int64_t)r * a.T + k0 + kk] = 0.f;
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (sm.abort_flag) {
    // give copies that may still be in flight time to land before the shared memory is released
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (wid == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------------
// Fused attention forward (Section 3.1, Eq. 1): out[j] = sum_{i<=j} a_i^j v_i and the row normalisers in
// ONE streaming sweep, so that a caller who needs the layer's output anyway pays a single further
// recomputation of QK^T (pass 2 above) for the indicator - the cost the Limitations section ("FlashAttention
// Support for H2O") asks to remove.  It stands in for pass 1: same normalisers, same workspace layout.
//
//   per work item (unit, tile of 128 queries), streamed key / value chunks of 128 tokens 0 .. diagonal:
//     S   = Q K^T            tcgen05, both operands K-major, fp32 in TMEM (two buffers)
//     P   = exp2(S - m)      two threads per query row, written back to TMEM as bf16 pairs (the A operand of the
//                            next product is read from there: P never touches shared memory, whose bandwidth
//                            the two products' operand reads and the incoming K and V tiles already use up)
//     O  += P V              tcgen05, V straight from its [token, d] rows as an MN-major B operand, O in TMEM
//     out = O / l, lse = m + log2 l
//   m is a per-row reference that follows the running maximum lazily: O and l are rescaled only when the
//   maximum has grown by more than 2^8 since the reference was set (probabilities stay below 2^8, far
//   inside bf16 and fp32 range; once the first chunks - which hold the attention sinks - are past, almost
//   no chunk rescales).  A rescale is a TMEM load / multiply / store of the thread's own row, done after
//   the previous P V product has completed and before this chunk's product is released.
// Warp roles (384 threads): warp 0 TMA producer and work-item FIFO, warp 1 issues S = Q K^T, warps 2-9 softmax (row =
// TMEM lane; two threads per row, 64 keys each, so that every scheduler has two warps to alternate between), warp 10
// value norms (Eq. 4), warp 11 issues O += P V.  The two products have an issuing thread each: they share no
// accumulator, every hand-over between them goes through the softmax warps' barriers, and one thread issuing both
// spent most of a chunk's time inside its sixteen MMA instructions and the waits between them (the logits of chunk
// c + 1 are then ready long before the softmax warps have finished chunk c).
constexpr int FW_NSW = 8;               // softmax warps: two per quarter of the rows
constexpr int FW_THREADS = (2 + FW_NSW + 2) * 32;
#ifndef FW_POLY_MASK
#define FW_POLY_MASK 0x0            // of the four pairs of an 8-probability piece, those whose exponential runs on the FMA pipe
#endif
constexpr int FW_ST = 3;               // stages of K and of V in shared memory
constexpr int FW_PB = 2;               // P buffers in TMEM
constexpr int FW_O_COL = 2 * TILE;     // TMEM columns: S buffers at 0 and 128, O at 256,
constexpr int FW_P_COL = 3 * TILE;     // P buffers (bf16 pairs, 64 columns each) at 384 and 448
constexpr float FW_LAZY = 8.f;         // log2 of the growth of a row maximum that forces a rescale

struct FwdSmem {
  alignas(1024) unsigned char q[TILE_BYTES];
  alignas(1024) unsigned char k[FW_ST][TILE_BYTES];    // [d half][128 tokens][128 bytes]
  alignas(1024) unsigned char v[FW_ST][TILE_BYTES];    // [d half][128 tokens][128 bytes]
  alignas(8) uint64_t q_full, q_empty;
  uint64_t k_full[FW_ST], k_empty[FW_ST], v_full[FW_ST], v_empty[FW_ST];
  uint64_t s_full[2], s_empty[2], p_full[FW_PB], p_empty[FW_PB];
  uint64_t o_full, o_empty;
  uint64_t item_full[4], item_empty[4];
  uint64_t pair_bar[4];                 // softmax warps q and q + 4 (same rows, other keys)
  int item_ring[4][2];                  // u, tile (u < 0: no more items)
  float lsum[2][TILE];                  // per key half: the row sums, exchanged at the end of an item
  uint32_t tmem_base;
  int abort_flag;
};

static_assert(sizeof(FwdSmem) + 1024 <= 227 * 1024, "the forward kernel's shared memory (with alignment slack) must fit one CTA");

// Shared-memory matrix descriptor of a V chunk as the B operand of O += P V: N (= d) is the contiguous
// dimension.  128-byte swizzle; a row of 64 d-values per token, 8 tokens per 1024-byte group (stride
// offset), the second 64 d-values one slab further on (leading offset).
__device__ __forceinline__ uint64_t umma_desc_mn(uint32_t smem_addr) {
  return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | ((uint64_t)(SLAB_BYTES >> 4) << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
constexpr uint32_t IDESC_PV = idesc<128>() | (1u << 16);   // B operand MN-major

__device__ __forceinline__ void umma_bf16_rt(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t id, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(id), "r"(acc)
      : "memory");
}
// the same with the A operand in TMEM: lane = row, 16-bit elements packed two to a column (K = 16 is 8 columns)
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t id, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(id), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t addr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(addr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
        "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
        "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
        "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
  const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);     // .x = lo is the lower address
  return *reinterpret_cast<const uint32_t*>(&t);
}

__global__ void __launch_bounds__(FW_THREADS, 1)
attention_fwd_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, TcArgs a, __nv_bfloat16* __restrict__ out) {
  extern __shared__ unsigned char smem_raw[];
  FwdSmem& sm = *reinterpret_cast<FwdSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  volatile int* abort_flag = &sm.abort_flag;
  const int items = a.units * a.nt;

  if (tid == 0) {
    mbar_init(&sm.q_full, 1); mbar_init(&sm.q_empty, 1);
    for (int i = 0; i < FW_ST; ++i) {
      mbar_init(&sm.k_full[i], 1); mbar_init(&sm.k_empty[i], 1);
      mbar_init(&sm.v_full[i], 1); mbar_init(&sm.v_empty[i], 1);
    }
    for (int i = 0; i < FW_PB; ++i) { mbar_init(&sm.p_full[i], FW_NSW); mbar_init(&sm.p_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sm.s_full[i], 1); mbar_init(&sm.s_empty[i], FW_NSW); }
    mbar_init(&sm.o_full, 1); mbar_init(&sm.o_empty, FW_NSW);
    for (int i = 0; i < 4; ++i) mbar_init(&sm.pair_bar[i], 2);
    for (int i = 0; i < 4; ++i) { mbar_init(&sm.item_full[i], 1); mbar_init(&sm.item_empty[i], 2 + FW_NSW); }   // two MMA warps + softmax warps
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (wid == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(&sm.tmem_base)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  if (a.wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");     // see reset_counters_kernel
  // pass 2, a programmatic dependent, may set up while this kernel runs
  if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // the itl-th item of this CTA: (u, tile), u < 0 ends the kernel (also when the CTA is aborting)
  auto next_item = [&](uint32_t itl, bool whole_warp, int& u, int& tile) {
    const int slot = itl & 3;
    bool got = mbar_wait(&sm.item_full[slot], (itl >> 2) & 1, abort_flag, a.dev_status);
    if (whole_warp) got = __all_sync(0xffffffffu, got);
    u = -1; tile = 0;
    if (got) {
      const volatile int* f = &sm.item_ring[slot][0];
      u = f[0]; tile = f[1];
    }
    if (whole_warp) __syncwarp();
    if (got && (!whole_warp || lane == 0)) mbar_arrive(&sm.item_empty[slot]);
  };

  if (wid == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      uint32_t n = 0;
      int next = (int)atomicAdd(&a.counters[0], 1u);
      for (uint32_t itl = 0; ok; ++itl) {
        const int id = next;
        const int slot = itl & 3;
        int u = -1, tile = 0;
        if (id < items) {
          // units in groups whose K, V and Q stay in L2 together; inside a group, longest items first
          const int grp = id / (a.gu * a.nt);
          const int rem = id - grp * (a.gu * a.nt);
          const int u0 = grp * a.gu;
          const int nu = min(a.gu, a.units - u0);
          const int r = rem / nu;
          u = u0 + (rem - r * nu);
          tile = a.nt - 1 - r;
        }
        ok = mbar_wait<20>(&sm.item_empty[slot], ((itl >> 2) & 1) ^ 1, abort_flag, a.dev_status);
        if (!ok) break;
        {
          volatile int* f = &sm.item_ring[slot][0];
          f[0] = u; f[1] = tile;
        }
        mbar_arrive(&sm.item_full[slot]);
        if (id >= items) break;
        next = (int)atomicAdd(&a.counters[0], 1u);
        const int b = u / a.heads, h = u - b * a.heads;
        ok = mbar_wait<20>(&sm.q_empty, (itl & 1) ^ 1, abort_flag, a.dev_status);
        if (!ok) break;
        mbar_expect_tx(&sm.q_full, TILE_BYTES);
        tma_load_4d(sm.q, &tm_q, &sm.q_full, 0, tile * TILE, h, b);
        tma_load_4d(sm.q + SLAB_BYTES, &tm_q, &sm.q_full, 64, tile * TILE, h, b);
        for (int c = 0; c <= tile; ++c, ++n) {
          const int stg = n % FW_ST;
          const uint32_t par = ((n / FW_ST) & 1) ^ 1;
          ok = mbar_wait<20>(&sm.k_empty[stg], par, abort_flag, a.dev_status);
          if (!ok) break;
          mbar_expect_tx(&sm.k_full[stg], TILE_BYTES);     // tokens beyond T arrive as zeros
          const int hk = a.G > 1 ? h / a.G : h;      // grouped queries: the KV head of this query head
          tma_load_4d(sm.k[stg], &tm_k, &sm.k_full[stg], 0, c * TILE, hk, b);
          tma_load_4d(sm.k[stg] + SLAB_BYTES, &tm_k, &sm.k_full[stg], 64, c * TILE, hk, b);
          ok = mbar_wait<20>(&sm.v_empty[stg], par, abort_flag, a.dev_status);
          if (!ok) break;
          mbar_expect_tx(&sm.v_full[stg], TILE_BYTES);
          tma_load_4d(sm.v[stg], &tm_v, &sm.v_full[stg], 0, c * TILE, hk, b);
          tma_load_4d(sm.v[stg] + SLAB_BYTES, &tm_v, &sm.v_full[stg], 64, c * TILE, hk, b);
        }
      }
    }
  } else if (wid == 1) {
    // ------------------------------------------------------------------ MMA issuer: S = Q K^T
    if (lane == 0) {
      bool ok = true;
      uint32_t n = 0;
      const uint64_t q_desc = umma_desc(s32(sm.q));
      const uint64_t k_desc0 = umma_desc(s32(sm.k[0]));
      // S(g) = Q K(g)^T into S buffer g % 2
      auto issue_qk = [&](uint32_t g) -> bool {
        const int stg = g % FW_ST, sb = g & 1;
        if (!mbar_wait(&sm.k_full[stg], (g / FW_ST) & 1, abort_flag, a.dev_status) ||
            !mbar_wait(&sm.s_empty[sb], ((g >> 1) & 1) ^ 1, abort_flag, a.dev_status))
          return false;
        tc_fence_after();
        const uint64_t kd = k_desc0 + (uint64_t)stg * (TILE_BYTES >> 4);
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk)
          umma_bf16_rt(tmem + sb * TILE, q_desc + k_off_fixed(kk), kd + k_off_fixed(kk), idesc<128>(), kk > 0);
        umma_commit(&sm.k_empty[stg]);
        umma_commit(&sm.s_full[sb]);
        return true;
      };
      for (uint32_t itl = 0; ok; ++itl) {
        int u, tile;
        next_item(itl, false, u, tile);
        if (u < 0) break;
        if (!VATP_INB(u, a.units, a.dev_status) || !VATP_INB(tile, a.nt, a.dev_status)) break;
        ok = mbar_wait(&sm.q_full, itl & 1, abort_flag, a.dev_status);
        if (!ok) break;
        const int nc = tile + 1;
        for (int c = 0; c < nc && ok; ++c) ok = issue_qk(n + c);
        if (ok) umma_commit(&sm.q_empty);            // the item's last S has been issued: the query tile may be replaced
        n += nc;
      }
    }
  } else if (wid == 3 + FW_NSW) {
    // ------------------------------------------------------------------ second MMA issuer: O += P V
    if (lane == 0) {
      bool ok = true;
      uint32_t n = 0;
      const uint64_t v_desc0 = umma_desc_mn(s32(sm.v[0]));
      for (uint32_t itl = 0; ok; ++itl) {
        int u, tile;
        next_item(itl, false, u, tile);
        if (u < 0) break;
        if (!VATP_INB(u, a.units, a.dev_status) || !VATP_INB(tile, a.nt, a.dev_status)) break;
        const int nc = tile + 1;
        for (int c = 0; c < nc && ok; ++c) {
          const uint32_t g = n + c;
          const int stg = g % FW_ST, pb = g % FW_PB;
          ok = mbar_wait(&sm.p_full[pb], (g / FW_PB) & 1, abort_flag, a.dev_status) &&
               mbar_wait(&sm.v_full[stg], (g / FW_ST) & 1, abort_flag, a.dev_status) &&
               (c > 0 || mbar_wait(&sm.o_empty, (itl & 1) ^ 1, abort_flag, a.dev_status));
          if (!ok) break;
          tc_fence_after();
          const uint64_t vd = v_desc0 + (uint64_t)stg * (TILE_BYTES >> 4);
#pragma unroll
          for (int kk = 0; kk < TILE / 16; ++kk)      // 16 keys per step: 8 columns further on in P, 2048 bytes in V
            umma_bf16_ts(tmem + FW_O_COL, tmem + FW_P_COL + pb * 64 + kk * 8, vd + (uint64_t)(kk * 128), IDESC_PV,
                         (c > 0 || kk > 0) ? 1u : 0u);
          umma_commit(&sm.v_empty[stg]);
          umma_commit(&sm.p_empty[pb]);
          if (c == nc - 1) umma_commit(&sm.o_full);
        }
        n += nc;
      }
    }
  } else if (wid < 2 + FW_NSW) {
    // ------------------------------------------------------------------ softmax: two threads per query row
    const int quarter = wid & 3;                  // TMEM lanes this warp may touch
    const int half = (wid - 2) >> 2;              // which 64 of a chunk's 128 keys (and of O's 128 columns) are this thread's
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16) + half * 64;
    const float sc = a.scale_log2;
    bool ok = true;
    uint32_t n = 0;
    // the two warps that share a quarter of the rows meet at an mbarrier of their own (a bounded wait like all
    // others: one arrival per warp, after which the partner's shared-memory stores are visible)
    uint32_t pair_phase = 0;
    auto pair_sync = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.pair_bar[quarter]);
      bool got = mbar_wait(&sm.pair_bar[quarter], pair_phase & 1, abort_flag, a.dev_status);
      ++pair_phase;
      return __all_sync(0xffffffffu, got);
    };
    for (uint32_t itl = 0; ok; ++itl) {
      int u, tile;
      next_item(itl, true, u, tile);
      if (u < 0) break;
      if (!VATP_INB(u, a.units, a.dev_status) || !VATP_INB(tile, a.nt, a.dev_status)) break;
      const int tok = tile * TILE + row;
      const int nc = tile + 1;
      float m_ref = -INFINITY, l_run = 0.f;       // l_run: this thread's 64 columns only
      for (int c = 0; c < nc; ++c) {
        const uint32_t g = n + c;
        const int sb = g & 1, pb = g % FW_PB;
        bool w = mbar_wait(&sm.s_full[sb], (g >> 1) & 1, abort_flag, a.dev_status);
        w = __all_sync(0xffffffffu, w);
        if (!w) { ok = false; break; }
        tc_fence_after();
        // own 64 columns (kept), then the partner's 64 for the row maximum only: reading them from TMEM
        // again costs less than an exchange through shared memory and a rendezvous in every chunk
        float x[2][32];
        float mx;
        {
          float y[2][32];
          const uint32_t other = lane_addr + sb * TILE + (half ? -64 : 64);
          tmem_ld32(lane_addr + sb * TILE, x[0]);
          tmem_ld32(lane_addr + sb * TILE + 32, x[1]);
          tmem_ld32(other, y[0]);
          tmem_ld32(other + 32, y[1]);
          tmem_ld_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.s_empty[sb]);
          if (c == tile) {
            mask_after_diagonal(x[0], half * 64, row);
            mask_after_diagonal(x[1], half * 64 + 32, row);
            mask_after_diagonal(y[0], (half ^ 1) * 64, row);
            mask_after_diagonal(y[1], (half ^ 1) * 64 + 32, row);
          }
          // scaled maximum of the row's 128 logits (scale > 0)
          mx = fmaxf(fmaxf(slice_max(x[0]), slice_max(x[1])), fmaxf(slice_max(y[0]), slice_max(y[1]))) * sc;
        }
        const float m_new = fmaxf(m_ref, mx);
        if (c == 0) {
          m_ref = m_new;              // finite: column 0 is never masked
        } else {
          const bool need = m_new > m_ref + FW_LAZY;
          if (__any_sync(0xffffffffu, need)) {
            // O += P(g-1) V(g-1) must have completed before this thread's part of its row of O is rewritten
            bool w2 = mbar_wait(&sm.p_empty[(g - 1) % FW_PB], ((g - 1) / FW_PB) & 1, abort_flag, a.dev_status);
            w2 = __all_sync(0xffffffffu, w2);
            if (!w2) { ok = false; break; }
            tc_fence_after();
            const float f = need ? ex2(m_ref - m_new) : 1.f;
#pragma unroll
            for (int q2 = 0; q2 < 2; ++q2) {
              float y[32];
              tmem_ld32(lane_addr + FW_O_COL + q2 * 32, y);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) y[i] *= f;
              tmem_st32(lane_addr + FW_O_COL + q2 * 32, y);
            }
            tmem_st_wait();
            l_run *= f;
            if (need) m_ref = m_new;
          }
        }
        // the P buffer is free once the product that read it two chunks ago has completed
        bool w3 = mbar_wait(&sm.p_empty[pb], ((g / FW_PB) & 1) ^ 1, abort_flag, a.dev_status);
        w3 = __all_sync(0xffffffffu, w3);
        if (!w3) { ok = false; break; }
        tc_fence_after();
        const f32x2 c2 = pk2(sc, sc), nm2 = pk2(-m_ref, -m_ref);
        f32x2 la = pk2(0.f, 0.f), lb = la;
        float pk[32];                              // 64 probabilities as bf16 pairs: this thread's columns of the P buffer
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float* xs = &x[j >> 2][(j & 3) * 8];
#pragma unroll
          for (int i = 0; i < 8; i += 2) {
            const f32x2 t = fma2(pk2(xs[i], xs[i + 1]), c2, nm2);
            const f32x2 e = ((FW_POLY_MASK >> (i >> 1)) & 1) ? ex2_fma2(t) : ex2_sfu2(t);
            if (i & 2) lb = add2(lb, e); else la = add2(la, e);
            float p0, p1;
            upk2(e, p0, p1);
            pk[j * 4 + (i >> 1)] = __uint_as_float(pack2_bf16(p0, p1));
          }
        }
        tmem_st32(tmem + ((uint32_t)(quarter * 32) << 16) + FW_P_COL + pb * 64 + half * 32, pk);
        l_run += hsum2(add2(la, lb));
        // P and any rescaled O (TMEM stores) are complete before the MMA warp is told
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.p_full[pb]);
      }
      if (!ok) break;
      n += nc;
      // ---- end of item: out = O / l, lse = m + log2 l (l: both halves of the row)
      sm.lsum[half][row] = l_run;
      if (!pair_sync()) { ok = false; break; }
      const float l_row = sm.lsum[0][row] + sm.lsum[1][row];
      if (!pair_sync()) { ok = false; break; }      // both have read: the next item may overwrite
      bool w4 = mbar_wait(&sm.o_full, itl & 1, abort_flag, a.dev_status);
      w4 = __all_sync(0xffffffffu, w4);
      if (!w4) { ok = false; break; }
      tc_fence_after();
      const float inv = 1.f / l_row;
      const int64_t o_off = (int64_t)(u / a.heads) * a.out_sb + (int64_t)(u % a.heads) * a.out_sh + (int64_t)tok * HD;
      __nv_bfloat16* orow = out + o_off + half * 64;
      const bool live = tok < a.T && VATP_INB(o_off, (int64_t)(a.units / a.heads) * a.out_sb, a.dev_status);
#pragma unroll
      for (int q2 = 0; q2 < 2; ++q2) {
        float y[32];
        tmem_ld32(lane_addr + FW_O_COL + q2 * 32, y);
        tmem_ld_wait();
        if (live) {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            reinterpret_cast<uint4*>(orow + q2 * 32)[j] =
                make_uint4(pack2_bf16(y[8 * j] * inv, y[8 * j + 1] * inv), pack2_bf16(y[8 * j + 2] * inv, y[8 * j + 3] * inv),
                           pack2_bf16(y[8 * j + 4] * inv, y[8 * j + 5] * inv), pack2_bf16(y[8 * j + 6] * inv, y[8 * j + 7] * inv));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.o_empty);
      if (half == 0) {
        const float lse2 = m_ref + log2f(l_row);
        // the layout pass 2 reads: negated, -inf where a query contributes nothing (beyond the prompt, before the
        // history window), half a chunk of padding after an odd tile count
        if (VATP_INB((int64_t)u * a.Tpad + tok, (int64_t)a.units * a.Tpad, a.dev_status))
          a.lse2[(int64_t)u * a.Tpad + tok] = (tok < a.T && tok >= a.first_row) ? -lse2 : -INFINITY;
        if ((a.nt & 1) && tile == a.nt - 1 && VATP_INB((int64_t)u * a.Tpad + tok + TILE, (int64_t)a.units * a.Tpad, a.dev_status))
          a.lse2[(int64_t)u * a.Tpad + tok + TILE] = -INFINITY;
        if (a.lse_out && tok < a.T)
          a.lse_out[(int64_t)(u / a.heads) * a.lse_sb + (int64_t)(u % a.heads) * a.lse_sh + tok] = lse2 * 0.69314718055994531f;
      }
    }
  } else if (a.side_norm) {
    // ------------------------------------------------------------------ value norms (Eq. 4)
    side_value_norms<VATP_NORM_L1>(a, lane);
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (sm.abort_flag) {
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (wid == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

// Zeroes the two work-item counters.  Launched as a programmatic dependent, with pass 1 as its own dependent: both
// are resident early and the launch latencies of a scoring call that follows other work on the stream are hidden;
// nothing is written before everything earlier in the stream has completed.
__global__ void reset_counters_kernel(unsigned* counters) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (threadIdx.x < 2) counters[threadIdx.x] = 0u;
}

// Value norms as a kernel of their own (Eq. 4): used with a history window, where pass 1 covers only
// the window's query tiles and is too short to hide one warp per SM walking all of V, and for the
// l2 / l-infinity variants.  Sixteen lanes
// per row, eight rows in flight per lane.
// When the caller supplies the row normalisers (lse_in, natural log, [units][T]) the same launch brings them
// into the layout pass 2 reads and so stands in for pass 1: log2 domain and negated, padded to whole chunks,
// -inf where a query contributes nothing (beyond the prompt, before the history window).
template <int KIND>
__global__ void __launch_bounds__(256) vnorm_kernel(TcArgs a, const float* __restrict__ lse_in) {
  // pass 2, a programmatic dependent, may set up while this kernel runs; it reads what is written here
  // only after its griddepcontrol.wait
  if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int u = blockIdx.x;
  if (lse_in) {
    // this CTA's 128 tokens; the last CTA of the unit also fills the padding up to Tpad
    const int last = blockIdx.y == gridDim.y - 1 ? a.Tpad : (blockIdx.y + 1) * 128;
    for (int i = blockIdx.y * 128 + threadIdx.x; i < last; i += 256) {
      float x = -INFINITY;
      if (i < a.T) {
        const float l = __ldg(lse_in + (int64_t)u * a.T + i);
        if (i >= a.first_row) x = -l * 1.4426950408889634f;
        if (a.lse_out && a.lse_out != lse_in) a.lse_out[(int64_t)u * a.T + i] = l;
      }
      a.lse2[(int64_t)u * a.Tpad + i] = x;
    }
  }
  const int b = u / a.kv_heads, h = u - b * a.kv_heads;      // (one CTA column per KV unit)
  const __nv_bfloat16* vu = a.v + (int64_t)b * a.sb + (int64_t)h * a.sh;
  const int sub = threadIdx.x >> 4, part = threadIdx.x & 15;       // 16 rows per pass of the CTA
  const int row0 = blockIdx.y * 128 + sub;
  uint4 raw[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int tok = row0 + 16 * j;
    raw[j] = make_uint4(0u, 0u, 0u, 0u);
    if (tok < a.T) raw[j] = __ldg(reinterpret_cast<const uint4*>(vu + (int64_t)tok * a.st) + part);
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t w[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i)
      acc = norm_fold(KIND, norm_fold(KIND, acc, __uint_as_float(w[i] << 16)), __uint_as_float(w[i] & 0xffff0000u));
#pragma unroll
    for (int o = 8; o; o >>= 1) acc = norm_merge(KIND, acc, __shfl_xor_sync(0xffffffffu, acc, o));
    const int tok = row0 + 16 * j;
    if (part == 0 && tok < a.T) a.vnorm[(int64_t)u * a.T + tok] = norm_finish(KIND, acc);
  }
}


// ---- history-window state from Q and the compacted keys (Eq. 3) ------------------------------------------
// For the kept tokens of a unit, their probabilities under the last w prompt queries, written in the layout the
// decode step keeps (ring[u][j mod w][slot]) together with the exact fixed-point sum per slot:
//   p[j][slot] = exp2(scale_log2 * <q_j, k_slot> - lse2_j)   for pos[slot] <= j (causal), else 0
// One CTA takes 128 slots of a unit (TMEM lanes = keys, as in pass 2) against the window's queries in chunks
// of 256 (accumulator columns): S^T = K_kept Q_win^T is one 128 x 256 x 128 block of MMAs per chunk.  Sixteen
// warps read it back: warp (quarter, group) takes 32 slots (one per thread) and 64 of the chunk's queries, so
// a slot's window sum is a running sum in four threads' registers (added up at the end; integers, so the order
// is immaterial), and for each query the 32 lanes of a warp store 32 consecutive slots of one ring row.
constexpr int RG_THREADS = 512;
struct RingSmem {
  alignas(1024) unsigned char keys[TILE_BYTES];     // 128 cached keys: two K halves of [128 rows][128 bytes]
  alignas(1024) unsigned char qrows[CHUNK_BYTES];   // 256 window queries: [K half][256 rows][128 bytes]
  float nlse[CHUNK];                                // their negated log2 normalisers (-inf: no such query)
  long long part[3][TILE];                          // window sums of column groups 1-3
  alignas(8) uint64_t bar_ld, bar_mma;
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(RG_THREADS, 2)
window_ring_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kc, int heads, int T,
                      int w, int B, int cap, float scale_log2, const float* __restrict__ lse, vatp_cache c,
                      int32_t* dev_status) {
  extern __shared__ unsigned char smem_raw[];
  RingSmem& sm = *reinterpret_cast<RingSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int u = blockIdx.y, slot0 = blockIdx.x * TILE;
  const int b = u / heads, h = u - b * heads;
  volatile int* abort_flag = &sm.abort_flag;
  if (tid == 0) {
    mbar_init(&sm.bar_ld, 1);
    mbar_init(&sm.bar_mma, 1);
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (wid == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(&sm.tmem_base)), "r"(CHUNK) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  const int quarter = wid & 3, grp = wid >> 2;      // TMEM lanes this warp may touch; which 64 columns of a chunk it takes
  const int row = quarter * 32 + lane;
  const int slot = slot0 + row;                     // this thread's slot = its TMEM lane
  const int len = min(T, B);
  const int ps = slot < len ? c.pos[(int64_t)u * cap + slot] : -1;      // position of the cached token, -1: empty slot
  float* ring_s = c.ring + (int64_t)u * w * cap + slot;     // this slot's column of the unit's ring
  long long fx = 0;
  bool ok = true;
  uint32_t it = 0;
  for (int c0 = 0; c0 < w && ok; c0 += CHUNK, ++it) {
    // the previous chunk's accumulator and normalisers have been consumed by every warp
    tc_fence_before();
    __syncthreads();
    for (int i = tid; i < CHUNK; i += RG_THREADS) {
      const int r = c0 + i, j = T - w + r;
      sm.nlse[i] = (r < w && j >= 0) ? -__ldg(lse + (int64_t)u * T + j) * 1.4426950408889634f : -INFINITY;
    }
    if (tid == 0) {
      mbar_expect_tx(&sm.bar_ld, CHUNK_BYTES + (it == 0 ? TILE_BYTES : 0));
      if (it == 0) {
        tma_load_2d(sm.keys, &tm_kc, &sm.bar_ld, 0, u * cap + slot0);
        tma_load_2d(sm.keys + SLAB_BYTES, &tm_kc, &sm.bar_ld, 64, u * cap + slot0);
      }
      // rows before the prompt (negative coordinate) and beyond it arrive as zeros
#pragma unroll
      for (int kh = 0; kh < 2; ++kh)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
          tma_load_4d(sm.qrows + kh * (2 * SLAB_BYTES) + hh * SLAB_BYTES, &tm_q, &sm.bar_ld, 64 * kh, T - w + c0 + hh * TILE, h, b);
      if (mbar_wait(&sm.bar_ld, it & 1, abort_flag, dev_status)) {
        tc_fence_after();
        umma_tile<0, 256>(tmem, umma_desc(s32(sm.keys)), umma_desc(s32(sm.qrows)));
        umma_commit(&sm.bar_mma);
      }
    }
    __syncthreads();                                 // normalisers written (thread 0 has issued the MMAs or given up)
    const bool got = mbar_wait(&sm.bar_mma, it & 1, abort_flag, dev_status);
    if (!__syncthreads_and(got ? 1 : 0)) { ok = false; break; }     // the same verdict for every warp of the CTA
    tc_fence_after();
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    const int n_cols = min(CHUNK, w - c0);
    for (int cs = 64 * grp; cs < min(n_cols, 64 * grp + 64); cs += 32) {
      float x[32];
      tmem_ld32(lane_addr + cs, x);
      tmem_ld_wait();
      // window row r = c0 + cs + i is query j = T - w + r and ring row j mod w; both advance by one per column
      // (the ring row wraps at w; -w < j < 0 when the prompt is shorter than the window)
      const int j0 = T - w + c0 + cs;
      int rr = j0 >= 0 ? j0 % w : j0 + w;
      uint32_t off = (uint32_t)rr * (uint32_t)cap;          // element offset of the ring row (w * cap < 2^31: checked on the host)
      const int live = min(32, n_cols - cs);
      const uint32_t lp = s32(&sm.nlse[cs]);
      if (live == 32 && rr + 32 <= w) {
        // the common case - a whole wave inside the window, no wrap of the ring row inside it: no per-column
        // bookkeeping.  Column i is visible to this slot's token iff ps <= j0 + i, i.e. i >= first (-1 < first: ps >= 0).
        const int first = ps >= 0 ? max(ps - j0, 0) : 32;
        const bool st_ok = slot < cap;
        float* out_p = ring_s + off;
#pragma unroll
        for (int i4 = 0; i4 < 32; i4 += 4) {
          float4 nl;
          asm("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(nl.x), "=f"(nl.y), "=f"(nl.z), "=f"(nl.w) : "r"(lp + 4 * i4));
          const float nls[4] = {nl.x, nl.y, nl.z, nl.w};
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int i = i4 + k;
            const float pr = i >= first ? ex2(fmaf(x[i], scale_log2, nls[k])) : 0.f;
            fx += prob_to_fixed(pr);
            if (st_ok && VATP_INB(off + (uint32_t)i * (uint32_t)cap, (int64_t)w * cap, dev_status)) out_p[(size_t)i * cap] = pr;
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (i < live) {
            float nl;
            asm("ld.shared.f32 %0, [%1];" : "=f"(nl) : "r"(lp + 4 * i));
            float pr = 0.f;
            if (ps >= 0 && ps <= j0 + i) pr = ex2(fmaf(x[i], scale_log2, nl));
            fx += prob_to_fixed(pr);
            if (slot < cap && VATP_INB(off, (int64_t)w * cap, dev_status)) ring_s[off] = pr;
            off += cap;
            if (++rr == w) { rr = 0; off = 0; }
          }
        }
      }
    }
  }
  if (grp > 0) sm.part[grp - 1][row] = fx;
  __syncthreads();
  if (ok && grp == 0 && slot < cap) {
    fx += sm.part[0][row] + sm.part[1][row] + sm.part[2][row];
    c.acc_fixed[(int64_t)u * cap + slot] = fx;
    c.acc[(int64_t)u * cap + slot] = fixed_to_prob(fx);
  }
  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (sm.abort_flag) {
    for (int i = 0; i < 200; ++i) __nanosleep(1000);   // copies that may still be in flight
    __syncthreads();
  }
  if (wid == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(CHUNK) : "memory");
  }
}

// ---- host side -------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// [batch, heads, T, 128] bf16 with element strides (sb, sh, st, 1); box = 64 x 128 rows, 128-byte swizzle
bool make_map(CUtensorMap* m, const void* base, const Shape& s, bool of_q = false) {
  const int heads = (!of_q && s.kv_heads > 0) ? s.kv_heads : s.heads;      // k and v of grouped queries: the KV heads
  const cuuint64_t dims[4] = {(cuuint64_t)HD, (cuuint64_t)s.T, (cuuint64_t)heads, (cuuint64_t)(s.units / s.heads)};
  const cuuint64_t strides[3] = {(cuuint64_t)s.st * 2, (cuuint64_t)(of_q ? s.qsh : s.sh) * 2, (cuuint64_t)(of_q ? s.qsb : s.sb) * 2};
  const cuuint32_t box[4] = {64, TILE, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool make_rows_map_bf16(CUtensorMap* m, const void* base, uint64_t rows, uint32_t box_rows) {
  if (!encode_fn()) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)HD, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)HD * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_row_gather_map(CUtensorMap* m, const void* base, uint32_t row_words, uint64_t rows, uint64_t row_stride_bytes) {
  if (!encode_fn()) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)row_words, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)row_stride_bytes};
  const cuuint32_t box[2] = {row_words, 1};
  const cuuint32_t estr[2] = {1, 1};
  return encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Per-device facts, looked up on first use with that device current (a process may drive several GPUs).
namespace {
constexpr int kMaxDevices = 64;
struct DeviceFacts {
  int known, tc, sms;
};
DeviceFacts g_facts[kMaxDevices];
std::mutex g_facts_mutex;

DeviceFacts device_facts() {
  int dev = 0;
  DeviceFacts f{1, 0, 148};
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return f;
  std::lock_guard<std::mutex> lock(g_facts_mutex);
  if (!g_facts[dev].known) {
    int major = 0, sms = 0;
    f.tc = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess && major == 10 &&
           encode_fn() != nullptr;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) f.sms = sms;
    g_facts[dev] = f;
  }
  return g_facts[dev];
}
}  // namespace

bool vatp_tc_available() { return device_facts().tc == 1; }
int device_sm_count() { return device_facts().sms; }

size_t prefill_tc_workspace_bytes(int units, int T) {
  const size_t Tpad = (size_t)(T + CHUNK - 1) / CHUNK * CHUNK;
  return ((size_t)units * Tpad * sizeof(float) + 255) / 256 * 256 + 256;   // normalisers, then the work-item counters
}

cudaError_t launch_prefill_tc(const Shape& s, const void* q, const void* k, const void* v, float* lse_ws,
                              float* lse_out, float* attn_acc, float* vnorm, float* score, float* win_rows,
                              int32_t* dev_status, cudaStream_t st, const float* lse_in, void* attn_out) {
  CUtensorMap tm_q, tm_k, tm_v;
  if (!make_map(&tm_q, q, s, true) || !make_map(&tm_k, k, s)) return cudaErrorInvalidValue;
  if (attn_out && (lse_in || !make_map(&tm_v, v, s))) return cudaErrorInvalidValue;
  TcArgs a;
  a.units = s.units; a.heads = s.heads; a.T = s.T;
  a.kv_heads = s.kv_heads > 0 ? s.kv_heads : s.heads;
  a.G = s.heads / a.kv_heads;
  a.kv_units = s.units / a.G;
  if (a.G > 1 && (lse_in || win_rows)) return cudaErrorInvalidValue;
  a.nt = (s.T + TILE - 1) / TILE;
  a.nch = (a.nt + 1) / 2;
  a.Tpad = a.nch * CHUNK;
  a.scale_log2 = s.scale * 1.4426950408889634f;
  a.v = static_cast<const __nv_bfloat16*>(v);
  a.sb = s.sb; a.sh = s.sh; a.st = s.st;
  a.lse_sb = s.lse_sb; a.lse_sh = s.lse_sh;
  a.out_sb = s.osb; a.out_sh = s.osh;
  a.lse2 = lse_ws; a.lse_out = lse_out; a.attn_acc = attn_acc; a.vnorm = vnorm; a.score = score;
  a.dev_status = dev_status;
  a.norm = s.norm;
  a.counters = reinterpret_cast<unsigned*>(reinterpret_cast<char*>(lse_ws) + ((size_t)a.units * a.Tpad * sizeof(float) + 255) / 256 * 256);
  const bool win = s.window > 0;
  a.window = win ? s.window : 0;
  a.first_row = win && s.T > s.window ? s.T - s.window : 0;
  a.ft = a.first_row / TILE;
  a.wrow0 = win ? s.T - s.window : 0;
  a.win_rows = win ? win_rows : nullptr;
  // K and Q of one unit are 2 * T * 256 bytes; keep a group's working set near 48 MB (L2 is 126 MB),
  // or take all units at once when everything fits anyway
  {
    const size_t unit_bytes = (size_t)2 * s.T * HD * 2;
    if ((size_t)s.units * unit_bytes <= ((size_t)96 << 20)) a.gu = s.units;
    else {
      const size_t g = ((size_t)48 << 20) / unit_bytes;
      a.gu = g < 1 ? 1 : (g > (size_t)s.units ? s.units : (int)g);
    }
  }
  const size_t smem = sizeof(Smem) + 1024;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(prefill_tc_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(prefill_tc_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(prefill_tc_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  const int sms = device_sm_count();
  const int items1 = a.units * (a.nt - a.ft), items2 = a.units * a.nt;
  // the side warp belongs to pass 1 (too short under a history window) or to the fused forward (always all tiles)
  a.side_norm = (a.ft == 0 || attn_out) && a.norm == VATP_NORM_L1 && !lse_in;
  // The counters are zeroed first.  When pass 1 follows at once, a one-warp kernel does it and pass 1 is its
  // programmatic dependent (see reset_counters_kernel); otherwise a memset node.
  a.wait_first = (a.side_norm && !lse_in) ? 1 : 0;
  if (a.wait_first) {
    DependentLaunch dr(dim3(1), dim3(32), 0, st);
    if ((e = cudaLaunchKernelEx(&dr.cfg, reset_counters_kernel, a.counters)) != cudaSuccess) return e;
  } else if ((e = cudaMemsetAsync(a.counters, 0, 2 * sizeof(unsigned), st)) != cudaSuccess) {
    return e;
  }
  if (!a.side_norm) {
    const dim3 grid(a.kv_units, (s.T + 127) / 128);
    if (a.norm == VATP_NORM_L1) vnorm_kernel<VATP_NORM_L1><<<grid, 256, 0, st>>>(a, lse_in);
    else if (a.norm == VATP_NORM_L2) vnorm_kernel<VATP_NORM_L2><<<grid, 256, 0, st>>>(a, lse_in);
    else vnorm_kernel<VATP_NORM_LINF><<<grid, 256, 0, st>>>(a, lse_in);
  }
  if (attn_out) {
    // the forward sweep stands in for pass 1; it streams K and V, so a group's units share the L2 three ways
    const size_t fsmem = sizeof(FwdSmem) + 1024;
    if ((e = cudaFuncSetAttribute(attention_fwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fsmem)) != cudaSuccess) return e;
    TcArgs af = a;
    const size_t unit_bytes = (size_t)3 * s.T * HD * 2;
    if ((size_t)s.units * unit_bytes > ((size_t)96 << 20)) {
      const size_t g = ((size_t)48 << 20) / unit_bytes;
      af.gu = g < 1 ? 1 : (g > (size_t)s.units ? s.units : (int)g);
    }
    if (a.wait_first) {
      DependentLaunch df(dim3(items2 < sms ? items2 : sms), dim3(FW_THREADS), fsmem, st);
      if ((e = cudaLaunchKernelEx(&df.cfg, attention_fwd_tc_kernel, tm_q, tm_k, tm_v, af, static_cast<__nv_bfloat16*>(attn_out))) !=
          cudaSuccess)
        return e;
    } else {
      attention_fwd_tc_kernel<<<items2 < sms ? items2 : sms, FW_THREADS, fsmem, st>>>(tm_q, tm_k, tm_v, af,
                                                                                      static_cast<__nv_bfloat16*>(attn_out));
    }
  } else if (a.wait_first && !lse_in) {
    DependentLaunch d1(dim3(items1 < sms ? items1 : sms), dim3(TC_THREADS), smem, st);
    if ((e = cudaLaunchKernelEx(&d1.cfg, prefill_tc_kernel<1, false>, tm_q, tm_k, a)) != cudaSuccess) return e;
  } else if (!lse_in) {
    prefill_tc_kernel<1, false><<<items1 < sms ? items1 : sms, TC_THREADS, smem, st>>>(tm_q, tm_k, a);
  }
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(items2 < sms ? items2 : sms);
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // the probabilities of the window's rows are written only when the caller wants them
  return win && win_rows ? cudaLaunchKernelEx(&cfg, prefill_tc_kernel<2, true>, tm_q, tm_k, a)
                         : cudaLaunchKernelEx(&cfg, prefill_tc_kernel<2, false>, tm_q, tm_k, a);
}

// Window history from Q and the compacted keys on the tensor cores (bf16, head_dim 128); see window_ring_tc_kernel.
cudaError_t launch_window_ring_tc(const Shape& s, int B, const void* q, const float* lse, const vatp_cache& c,
                                  int32_t* dev_status, cudaStream_t st) {
  const int cap = cache_capacity(B);
  CUtensorMap tm_q, tm_kc;
  if (!make_map(&tm_q, q, s, true) || !make_rows_map_bf16(&tm_kc, c.k_cache, (uint64_t)s.units * cap, TILE)) return cudaErrorInvalidValue;
  if ((int64_t)s.window * cap >= ((int64_t)1 << 31)) return cudaErrorInvalidValue;
  const size_t smem = sizeof(RingSmem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(window_ring_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  window_ring_tc_kernel<<<dim3((cap + TILE - 1) / TILE, s.units), RG_THREADS, smem, st>>>(
      tm_q, tm_kc, s.heads, s.T, s.window, B, cap, s.scale * 1.4426950408889634f, lse, c, dev_status);
  return cudaGetLastError();
}

}  // namespace vatp
