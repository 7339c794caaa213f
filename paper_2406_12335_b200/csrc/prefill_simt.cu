// fp32 FMA prefill scoring: exact-product two-pass column sums of the causal softmax matrix.
//
// Pass 1 gives every query row its log-sum-exp (the normaliser of Eq. 1); pass 2 recomputes the
// logits tile by tile and adds exp(s - lse) into per-key sums (Eq. 2, or Eq. 3 when only the last
// w query rows count), fused with the value l1 norm and the Eq. 4 product.  This is the path for
// fp32 inputs (tensor cores would round the operands) and for shapes the tensor-core kernel does
// not take.  No float atomics: each CTA owns a tile of rows (pass 1) or of keys (pass 2).
#include "vatp_internal.cuh"

namespace vatp {
namespace {

constexpr int TILE = 64;      // queries or keys per CTA tile
constexpr int NTHREADS = 256; // 16 x 16 threads, 4 x 4 logits each

template <typename T>
__device__ __forceinline__ void load_tile(float* dst, int ld, const T* src, int64_t row_stride, int row0, int rows_valid,
                                          int d) {
  // dst[r][c] for r < TILE; rows beyond rows_valid are zero
  const int vec = d / 4;
  for (int i = threadIdx.x; i < TILE * vec; i += NTHREADS) {
    int r = i / vec, c4 = (i % vec) * 4;
    float x0 = 0.f, x1 = 0.f, x2 = 0.f, x3 = 0.f;
    if (r < rows_valid) {
      const T* p = src + (int64_t)(row0 + r) * row_stride + c4;
      x0 = to_f32(p[0]); x1 = to_f32(p[1]); x2 = to_f32(p[2]); x3 = to_f32(p[3]);
    }
    float* o = dst + r * ld + c4;
    o[0] = x0; o[1] = x1; o[2] = x2; o[3] = x3;
  }
}

// s[i][j] = <A[ty + 16 i], B[tx + 16 j]> for the thread's 4 x 4 micro-tile
__device__ __forceinline__ void micro_gemm(const float* As, const float* Bs, int ld, int d, int ty, int tx,
                                           float (&s)[4][4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
  for (int c = 0; c < d; ++c) {
    float a[4], b[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) a[i] = As[(ty + 16 * i) * ld + c];
#pragma unroll
    for (int j = 0; j < 4; ++j) b[j] = Bs[(tx + 16 * j) * ld + c];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) s[i][j] = fmaf(a[i], b[j], s[i][j]);
  }
}

// Pass 1: one CTA per (query tile, unit).  lse[j] over keys i <= j.
template <typename T>
__global__ void __launch_bounds__(NTHREADS) rowstats_kernel(Shape sh, const T* __restrict__ q, const T* __restrict__ k,
                                                            float* __restrict__ lse, int first_row) {
  extern __shared__ float smem[];
  const int ld = sh.d + 1;
  float* Qs = smem;
  float* Ks = smem + TILE * ld;
  const int u = blockIdx.y;
  const int q0 = first_row + blockIdx.x * TILE;
  if (q0 >= sh.T) return;
  const T* qu = q + unit_offset_q(sh, u);
  const T* ku = k + unit_offset(sh, u);
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;

  load_tile(Qs, ld, qu, sh.st, q0, min(TILE, sh.T - q0), sh.d);
  float m[4], l[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) { m[i] = -INFINITY; l[i] = 0.f; }

  const int last_key = min(q0 + TILE, sh.T);  // exclusive
  for (int k0 = 0; k0 < last_key; k0 += TILE) {
    __syncthreads();
    load_tile(Ks, ld, ku, sh.st, k0, min(TILE, sh.T - k0), sh.d);
    __syncthreads();
    float s[4][4];
    micro_gemm(Qs, Ks, ld, sh.d, ty, tx, s);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = q0 + ty + 16 * i;
      float tile_max = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int col = k0 + tx + 16 * j;
        s[i][j] = (col <= row) ? s[i][j] * sh.scale : -INFINITY;
        tile_max = fmaxf(tile_max, s[i][j]);
      }
      if (tile_max > -INFINITY) {
        const float m_new = fmaxf(m[i], tile_max);
        float add = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) add += expf(s[i][j] - m_new);
        l[i] = l[i] * expf(m[i] - m_new) + add;
        m[i] = m_new;
      }
    }
  }
  // merge the 16 threads (same ty, consecutive lanes) that share each row
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m[i], off);
      const float l2 = __shfl_xor_sync(0xffffffffu, l[i], off);
      const float mn = fmaxf(m[i], m2);
      if (mn > -INFINITY) {
        l[i] = l[i] * expf(m[i] - mn) + l2 * expf(m2 - mn);
        m[i] = mn;
      }
    }
    const int row = q0 + ty + 16 * i;
    if (tx == 0 && row < sh.T) lse[unit_offset_lse(sh, u) + row] = m[i] + logf(l[i]);
  }
}

// Pass 2: one CTA per (key tile, unit).  Column sums over query rows j >= max(first_row, k).
template <typename T>
__global__ void __launch_bounds__(NTHREADS)
colsum_kernel(Shape sh, const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
              const float* __restrict__ lse, float* __restrict__ attn_acc, float* __restrict__ vnorm,
              float* __restrict__ score, float* __restrict__ win_rows, int first_row) {
  extern __shared__ float smem[];
  const int ld = sh.d + 1;
  float* Qs = smem;
  float* Ks = smem + TILE * ld;
  float* lse_s = Ks + TILE * ld;        // [TILE]
  float* red = lse_s + TILE;            // [16][TILE]
  const int u = blockIdx.y;
  const int k0 = blockIdx.x * TILE;
  const T* qu = q + unit_offset_q(sh, u);
  const T* ku = k + unit_offset(sh, u);
  const T* vu = v + unit_offset(sh, u);
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
  const int keys_valid = min(TILE, sh.T - k0);

  load_tile(Ks, ld, ku, sh.st, k0, keys_valid, sh.d);
  float cs[4] = {0.f, 0.f, 0.f, 0.f};

  // query tiles are aligned to first_row so that window rows map to whole tiles
  int qstart = first_row;
  if (k0 > first_row) qstart = first_row + ((k0 - first_row) / TILE) * TILE;
  const int wrow0 = sh.T - sh.window;   // query position of win_rows row 0 (may be negative)
  float* wr = win_rows ? win_rows + (int64_t)u * sh.window * sh.T : nullptr;

  if (wr) {
    // rows of the window that lie entirely above this key tile (j < k0): zeros
    for (int j = max(first_row, 0); j < min(qstart, sh.T); ++j)
      for (int c = threadIdx.x; c < keys_valid; c += NTHREADS) wr[(int64_t)(j - wrow0) * sh.T + k0 + c] = 0.f;
    // rows before the first token (T < w)
    for (int r = 0; r < -wrow0; ++r)
      for (int c = threadIdx.x; c < keys_valid; c += NTHREADS) wr[(int64_t)r * sh.T + k0 + c] = 0.f;
  }

  for (int q0 = qstart; q0 < sh.T; q0 += TILE) {
    __syncthreads();
    const int rows_valid = min(TILE, sh.T - q0);
    load_tile(Qs, ld, qu, sh.st, q0, rows_valid, sh.d);
    if (threadIdx.x < TILE) lse_s[threadIdx.x] = threadIdx.x < rows_valid ? lse[unit_offset_lse(sh, u) + q0 + threadIdx.x] : 0.f;
    __syncthreads();
    float s[4][4];
    micro_gemm(Qs, Ks, ld, sh.d, ty, tx, s);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = q0 + ty + 16 * i;
      const float lr = lse_s[ty + 16 * i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int col = k0 + tx + 16 * j;
        float p = 0.f;
        if (row < sh.T && col <= row && col < sh.T) p = expf(s[i][j] * sh.scale - lr);
        cs[j] += p;
        if (wr && row < sh.T && col < sh.T) wr[(int64_t)(row - wrow0) * sh.T + col] = p;
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < 4; ++j) red[ty * TILE + tx + 16 * j] = cs[j];
  // value norms (Eq. 4): 4 threads per row
  float* vn_s = Qs;  // reuse
  __syncthreads();
  {
    const int r = threadIdx.x / 4, part = threadIdx.x % 4;
    float acc = 0.f;
    if (r < keys_valid) {
      const T* p = vu + (int64_t)(k0 + r) * sh.st;
      for (int c = part; c < sh.d; c += 4) acc = norm_fold(sh.norm, acc, to_f32(p[c]));
    }
    acc = norm_merge(sh.norm, acc, __shfl_xor_sync(0xffffffffu, acc, 1));
    acc = norm_merge(sh.norm, acc, __shfl_xor_sync(0xffffffffu, acc, 2));
    if (part == 0) vn_s[r] = norm_finish(sh.norm, acc);
  }
  __syncthreads();
  if (threadIdx.x < keys_valid) {
    float tot = 0.f;
#pragma unroll
    for (int t = 0; t < 16; ++t) tot += red[t * TILE + threadIdx.x];
    const int64_t o = (int64_t)u * sh.T + k0 + threadIdx.x;
    const float n1 = vn_s[threadIdx.x];
    attn_acc[o] = tot;
    vnorm[o] = n1;
    score[o] = tot * n1;
  }
}

template <typename T>
cudaError_t launch_t(const Shape& s, const T* q, const T* k, const T* v, float* lse, float* attn_acc, float* vnorm,
                     float* score, float* win_rows, cudaStream_t st, bool lse_given) {
  const int ld = s.d + 1;
  const size_t smem1 = sizeof(float) * 2 * TILE * ld;
  const size_t smem2 = smem1 + sizeof(float) * (TILE + 16 * TILE);
  cudaError_t e;
  e = cudaFuncSetAttribute(rowstats_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(colsum_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2);
  if (e != cudaSuccess) return e;
  const int first_row = s.window > 0 ? max(s.T - s.window, 0) : 0;
  const int qtiles = (s.T - first_row + TILE - 1) / TILE;
  const int ktiles = (s.T + TILE - 1) / TILE;
  if (!lse_given) rowstats_kernel<T><<<dim3(qtiles, s.units), NTHREADS, smem1, st>>>(s, q, k, lse, first_row);
  colsum_kernel<T><<<dim3(ktiles, s.units), NTHREADS, smem2, st>>>(s, q, k, v, lse, attn_acc, vnorm, score,
                                                                    s.window > 0 ? win_rows : nullptr, first_row);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prefill_simt(const Shape& s, int dtype, const void* q, const void* k, const void* v, float* lse,
                                float* attn_acc, float* vnorm, float* score, float* win_rows, cudaStream_t st,
                                bool lse_given) {
  if (dtype == VATP_F32)
    return launch_t<float>(s, (const float*)q, (const float*)k, (const float*)v, lse, attn_acc, vnorm, score, win_rows, st,
                           lse_given);
  return launch_t<__nv_bfloat16>(s, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, lse,
                                 attn_acc, vnorm, score, win_rows, st, lse_given);
}

}  // namespace vatp
