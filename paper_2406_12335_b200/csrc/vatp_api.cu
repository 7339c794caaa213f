// Host side of the C ABI: argument checks, workspace carving, dispatch to the kernels.
#include <cstring>

#include "vatp_internal.cuh"

using namespace vatp;

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

vatp_status check_params(const vatp_params* p, bool need_T) {
  if (!p) return VATP_ERR_INVALID_ARG;
  if (p->batch <= 0 || p->heads <= 0) return VATP_ERR_INVALID_ARG;
  if (need_T && p->seq_len <= 0) return VATP_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return VATP_ERR_UNSUPPORTED;
  if (p->dtype != VATP_BF16 && p->dtype != VATP_F32) return VATP_ERR_UNSUPPORTED;
  if (p->indicator != VATP_IND_H2O && p->indicator != VATP_IND_WINDOW) return VATP_ERR_UNSUPPORTED;
  if (p->indicator == VATP_IND_WINDOW && p->window_w <= 0) return VATP_ERR_INVALID_ARG;
  if (p->norm_kind != VATP_NORM_L1 && p->norm_kind != VATP_NORM_L2 && p->norm_kind != VATP_NORM_LINF) return VATP_ERR_UNSUPPORTED;
  if (p->budget <= 0 || p->n_sink < 0 || p->n_recent < 0) return VATP_ERR_INVALID_ARG;
  if ((int64_t)p->n_sink + p->n_recent > p->budget) return VATP_ERR_INVALID_ARG;
  if (!(p->scale > 0.f)) return VATP_ERR_INVALID_ARG;
  if (p->stride_b < 0 || p->stride_h < 0 || p->stride_t < 0) return VATP_ERR_INVALID_ARG;
  if (p->flags & ~(int32_t)VATP_FLAG_DECODE_OVERLAP) return VATP_ERR_INVALID_ARG;
  if (p->kv_heads < 0 || p->kv_heads > p->heads || (p->kv_heads && p->heads % p->kv_heads)) return VATP_ERR_INVALID_ARG;
  if (p->kv_heads && p->kv_heads < p->heads && (p->stride_b || p->stride_h || p->stride_t)) return VATP_ERR_INVALID_ARG;
  return VATP_OK;
}

// query heads per KV head (1: multi-head attention) and the number of KV heads
inline int group_of(const vatp_params* p) { return p->kv_heads > 0 ? p->heads / p->kv_heads : 1; }
inline int kv_heads_of(const vatp_params* p) { return p->kv_heads > 0 ? p->kv_heads : p->heads; }

// The units are the (batch, KV head) pairs.  With grouped queries (contiguous layouts only) q has G times as many
// heads.  The general kernels take one query head of every group per launch, i.e. q as a view with head stride
// G * T * d (the caller offsets the q pointer by g * T * d and the row-normaliser pointer by g * T); the tensor-core
// kernels take all query heads in one launch (Shape::kv_heads).
vatp_status make_shape(const vatp_params* p, Shape* s) {
  const int kvh = kv_heads_of(p), G = group_of(p);
  s->units = p->batch * kvh;
  s->heads = kvh;
  s->kv_heads = 0;
  s->T = p->seq_len;
  s->d = p->head_dim;
  s->st = p->stride_t ? p->stride_t : p->head_dim;
  s->sh = p->stride_h ? p->stride_h : (int64_t)p->seq_len * s->st;
  s->sb = p->stride_b ? p->stride_b : (int64_t)kvh * s->sh;
  s->qsh = (int64_t)G * s->sh;
  s->qsb = G > 1 ? (int64_t)p->heads * s->sh : s->sb;
  s->lse_sh = (int64_t)G * p->seq_len;
  s->lse_sb = (int64_t)p->heads * p->seq_len;
  s->osh = (int64_t)G * p->seq_len * p->head_dim;
  s->osb = (int64_t)p->heads * p->seq_len * p->head_dim;
  s->scale = p->scale;
  s->window = p->indicator == VATP_IND_WINDOW ? p->window_w : 0;
  s->norm = p->norm_kind;
  const int eb = p->dtype == VATP_F32 ? 4 : 2;
  if (s->st < s->d) return VATP_ERR_INVALID_ARG;
  if ((s->st * eb) % 16 || (s->sh * eb) % 16 || (s->sb * eb) % 16) return VATP_ERR_INVALID_ARG;
  return VATP_OK;
}

// row normalisers of pass 1, padded to whole 128-row tiles per unit; with grouped queries, then the G partial
// indicators [G][units][T] that the group mean is taken of
inline size_t lse_bytes(const vatp_params* p) {
  size_t n = prefill_tc_workspace_bytes(p->batch * p->heads, p->seq_len);      // (one row per query head)
  return (n + 255) / 256 * 256;
}
inline size_t workspace_need(const vatp_params* p) {
  const int G = group_of(p);
  size_t n = lse_bytes(p);
  if (G > 1) n += ((size_t)G * p->batch * kv_heads_of(p) * p->seq_len * sizeof(float) + 255) / 256 * 256;
  return n;
}

bool cache_ok(const vatp_cache* c, bool windowed) {
  if (!c || !c->k_cache || !c->v_cache || !c->acc || !c->vnorm || !c->pos || !c->len || !c->free_slot || !c->next_pos ||
      !c->last_slot)
    return false;
  if (!aligned16(c->k_cache) || !aligned16(c->v_cache) || !aligned16(c->acc) || !aligned16(c->vnorm) || !aligned16(c->pos))
    return false;
  if (windowed && (!c->ring || !c->acc_fixed)) return false;
  return true;
}

// The prefill entry points: lse_in == nullptr runs pass 1, otherwise the caller's normalisers replace it;
// attn_out != nullptr runs the attention forward in pass 1's place (it yields the same normalisers).
vatp_status prefill_impl(const vatp_params* p, const void* q, const void* k, const void* v, const float* lse_in,
                         float* lse_out, float* attn_acc, float* vnorm, float* score, float* win_rows, void* workspace,
                         size_t workspace_bytes, int32_t* dev_status, void* cuda_stream, void* attn_out = nullptr) {
  vatp_status s = check_params(p, true);
  if (s != VATP_OK) return s;
  if (!q || !k || !v || !attn_acc || !vnorm || !score) return VATP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v)) return VATP_ERR_INVALID_ARG;
  Shape sh;
  s = make_shape(p, &sh);
  if (s != VATP_OK) return s;
  const int G = group_of(p);
  if (G > 1 && (lse_in || win_rows)) return VATP_ERR_UNSUPPORTED;
  if (attn_out && (lse_in || !aligned16(attn_out))) return VATP_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < workspace_need(p) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return VATP_ERR_WORKSPACE;
  float* ws = static_cast<float*>(workspace);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  decode_history_forget(st);
  cudaError_t e;
  if (G > 1) {
    // Every query head's indicator goes to a slice of the workspace - head g of its group to slice g - then the mean
    // over the slices (fixed order) and Eq. 4.  General kernels: one query head of every KV group per round, the
    // multi-head kernels on strided views of q.
    const size_t n = (size_t)sh.units * sh.T;
    float* part = reinterpret_cast<float*>(static_cast<char*>(workspace) + lse_bytes(p));
    const int eb = p->dtype == VATP_F32 ? 4 : 2;
    const bool tc = p->dtype == VATP_BF16 && p->head_dim == 128 && vatp_tc_available();
    // the general kernel keeps its (natural-log) normalisers in the caller's layout: lse_out, or a scratch copy of
    // that layout at the head of the workspace when the caller wants none (it fits: G * units * T floats <= `part`)
    e = cudaSuccess;
    if (tc) {
      // tensor cores: ONE launch over all query heads; unit (b, h) reads KV head h / G, and pass 2 files its indicator
      // under slice h % G of the partial indicators
      Shape sq = sh;
      sq.units = p->batch * p->heads;
      sq.heads = p->heads;
      sq.kv_heads = kv_heads_of(p);
      sq.qsh = sh.sh;
      sq.qsb = (int64_t)p->heads * sh.sh;
      sq.lse_sh = sh.T;
      sq.lse_sb = (int64_t)p->heads * sh.T;
      sq.osh = (int64_t)sh.T * sh.d;
      sq.osb = (int64_t)p->heads * sh.T * sh.d;
      e = launch_prefill_tc(sq, q, k, v, ws, lse_out, part, vnorm, score, nullptr, dev_status, st, nullptr, attn_out);
    }
    for (int g = 0; g < G && e == cudaSuccess && !tc; ++g) {
      const char* qg = static_cast<const char*>(q) + (size_t)g * sh.sh * eb;
      float* lse_g = lse_out ? lse_out + (size_t)g * sh.T : nullptr;
      // the fused call: this round's query heads' rows of the attention output (head kvh * G + g of every KV group)
      void* out_g = attn_out ? static_cast<char*>(attn_out) + (size_t)g * sh.T * sh.d * eb : nullptr;
      if (tc) {
        e = launch_prefill_tc(sh, qg, k, v, ws, lse_g, part + g * n, vnorm, score, nullptr, dev_status, st, nullptr, out_g);
      } else {
        Shape sg = sh;
        float* lse_buf = lse_g;
        if (!lse_buf) { lse_buf = ws; sg.lse_sb = (int64_t)sh.heads * sh.T; sg.lse_sh = sh.T; }   // plain [units][T] scratch
        if (out_g) {
          e = launch_attention_fwd_general(sg, p->dtype, qg, k, v, out_g, lse_buf, st);
          if (e == cudaErrorNotSupported) return VATP_ERR_UNSUPPORTED;
          if (e == cudaSuccess) e = launch_prefill_simt(sg, p->dtype, qg, k, v, lse_buf, part + g * n, vnorm, score, nullptr, st, true);
        } else {
          e = launch_prefill_simt(sg, p->dtype, qg, k, v, lse_buf, part + g * n, vnorm, score, nullptr, st);
        }
      }
    }
    if (e == cudaSuccess) e = launch_group_mean(G, (int64_t)n, part, vnorm, attn_acc, score, st);
    return e == cudaSuccess ? VATP_OK : VATP_ERR_CUDA;
  }
  if (p->dtype == VATP_BF16 && p->head_dim == 128 && vatp_tc_available()) {
    e = launch_prefill_tc(sh, q, k, v, ws, lse_out, attn_acc, vnorm, score, win_rows, dev_status, st, lse_in, attn_out);
  } else if (attn_out) {
    // general path: the forward leaves natural-log normalisers where pass 2 reads them (the caller's array, or
    // the workspace in the same layout)
    float* lse_buf = lse_out ? lse_out : ws;
    e = launch_attention_fwd_general(sh, p->dtype, q, k, v, attn_out, lse_buf, st);
    if (e == cudaErrorNotSupported) return VATP_ERR_UNSUPPORTED;
    if (e == cudaSuccess) e = launch_prefill_simt(sh, p->dtype, q, k, v, lse_buf, attn_acc, vnorm, score, win_rows, st, true);
  } else if (lse_in) {
    // pass 2 of the general kernel reads natural-log normalisers [units][T] directly
    e = launch_prefill_simt(sh, p->dtype, q, k, v, const_cast<float*>(lse_in), attn_acc, vnorm, score, win_rows, st, true);
    if (e == cudaSuccess && lse_out && lse_out != lse_in)
      e = cudaMemcpyAsync(lse_out, lse_in, sizeof(float) * (size_t)sh.units * sh.T, cudaMemcpyDeviceToDevice, st);
  } else {
    e = launch_prefill_simt(sh, p->dtype, q, k, v, lse_out ? lse_out : ws, attn_acc, vnorm, score, win_rows, st);
  }
  return e == cudaSuccess ? VATP_OK : VATP_ERR_CUDA;
}

}  // namespace

extern "C" {

const char* vatp_status_string(vatp_status s) {
  switch (s) {
    case VATP_OK: return "ok";
    case VATP_ERR_INVALID_ARG: return "invalid argument";
    case VATP_ERR_UNSUPPORTED: return "unsupported configuration";
    case VATP_ERR_WORKSPACE: return "workspace too small or misaligned";
    case VATP_ERR_CUDA: return "CUDA error";
    case VATP_ERR_TIMEOUT: return "device-side wait ran out";
    case VATP_ERR_STATIC_SCRATCH: return "problem exceeds the library's built-in scratch array";
    case VATP_ERR_BOUNDS: return "a kernel computed an index outside its array (bounds-checking build)";
  }
  return "unknown status";
}

int32_t vatp_cache_capacity(int32_t budget) { return budget > 0 ? cache_capacity(budget) : 0; }

size_t vatp_workspace_bytes(const vatp_params* p) {
  if (check_params(p, true) != VATP_OK) return 0;
  return workspace_need(p);
}

vatp_status vatp_prefill_scores(const vatp_params* p, const void* q, const void* k, const void* v, float* lse_out,
                                float* attn_acc, float* vnorm, float* score, float* win_rows, void* workspace,
                                size_t workspace_bytes, int32_t* dev_status, void* cuda_stream) {
  return prefill_impl(p, q, k, v, nullptr, lse_out, attn_acc, vnorm, score, win_rows, workspace, workspace_bytes,
                      dev_status, cuda_stream);
}

vatp_status vatp_prefill_attention_scores(const vatp_params* p, const void* q, const void* k, const void* v, void* attn_out,
                                          float* lse_out, float* attn_acc, float* vnorm, float* score, float* win_rows,
                                          void* workspace, size_t workspace_bytes, int32_t* dev_status, void* cuda_stream) {
  if (!attn_out) return VATP_ERR_INVALID_ARG;
  return prefill_impl(p, q, k, v, nullptr, lse_out, attn_acc, vnorm, score, win_rows, workspace, workspace_bytes, dev_status,
                      cuda_stream, attn_out);
}

vatp_status vatp_prefill_scores_from_lse(const vatp_params* p, const void* q, const void* k, const void* v,
                                         const float* lse_in, float* lse_out, float* attn_acc, float* vnorm,
                                         float* score, float* win_rows, void* workspace, size_t workspace_bytes,
                                         int32_t* dev_status, void* cuda_stream) {
  if (!lse_in || !aligned16(lse_in)) return VATP_ERR_INVALID_ARG;
  return prefill_impl(p, q, k, v, lse_in, lse_out, attn_acc, vnorm, score, win_rows, workspace, workspace_bytes,
                      dev_status, cuda_stream);
}

vatp_status vatp_select(const vatp_params* p, const float* score, int32_t* kept_idx, void* workspace,
                        size_t workspace_bytes, int32_t* dev_status, void* cuda_stream) {
  (void)workspace; (void)workspace_bytes;
  vatp_status s = check_params(p, true);
  if (s != VATP_OK) return s;
  if (!score || !kept_idx) return VATP_ERR_INVALID_ARG;
  decode_history_forget(static_cast<cudaStream_t>(cuda_stream));
  cudaError_t e = launch_select(p->batch * kv_heads_of(p), p->seq_len, p->budget, p->n_sink, p->n_recent, score, kept_idx,
                                dev_status, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? VATP_OK : VATP_ERR_CUDA;
}

vatp_status vatp_compact(const vatp_params* p, const void* k, const void* v, const float* attn_acc,
                         const float* vnorm, const float* win_rows, const int32_t* kept_idx, const vatp_cache* cache,
                         int32_t* dev_status, void* cuda_stream) {
  vatp_status s = check_params(p, true);
  if (s != VATP_OK) return s;
  const bool windowed = p->indicator == VATP_IND_WINDOW;
  if (!k || !v || !attn_acc || !vnorm || !kept_idx || !cache_ok(cache, windowed)) return VATP_ERR_INVALID_ARG;
  if (windowed && !win_rows) return VATP_ERR_INVALID_ARG;
  if (windowed && group_of(p) > 1) return VATP_ERR_UNSUPPORTED;
  if (!aligned16(k) || !aligned16(v)) return VATP_ERR_INVALID_ARG;
  Shape sh;
  s = make_shape(p, &sh);
  if (s != VATP_OK) return s;
  decode_history_forget(static_cast<cudaStream_t>(cuda_stream));
  cudaError_t e = launch_compact(sh, p->dtype, p->budget, k, v, attn_acc, vnorm, win_rows, kept_idx, *cache,
                                 dev_status, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? VATP_OK : VATP_ERR_CUDA;
}

vatp_status vatp_compact_window(const vatp_params* p, const void* q, const void* k, const void* v, const float* lse,
                                const float* attn_acc, const float* vnorm, const int32_t* kept_idx,
                                const vatp_cache* cache, int32_t* dev_status, void* cuda_stream) {
  vatp_status s = check_params(p, true);
  if (s != VATP_OK) return s;
  if (p->indicator != VATP_IND_WINDOW) return VATP_ERR_INVALID_ARG;
  if (!q || !k || !v || !lse || !attn_acc || !vnorm || !kept_idx || !cache_ok(cache, true)) return VATP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v)) return VATP_ERR_INVALID_ARG;
  Shape sh;
  s = make_shape(p, &sh);
  if (s != VATP_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  decode_history_forget(st);
  cudaError_t e = launch_compact(sh, p->dtype, p->budget, k, v, attn_acc, vnorm, nullptr, kept_idx, *cache, dev_status, st);
  if (e == cudaSuccess)
    e = group_of(p) > 1 ? launch_window_ring_grouped(sh, group_of(p), p->dtype, p->budget, q, lse, *cache, st)
                        : launch_window_ring(sh, p->dtype, p->budget, q, lse, *cache, dev_status, st);
  return e == cudaSuccess ? VATP_OK : (e == cudaErrorNotSupported ? VATP_ERR_UNSUPPORTED : VATP_ERR_CUDA);
}

vatp_status vatp_decode_step(const vatp_params* p, const vatp_cache* cache, const void* q_new, const void* k_new,
                             const void* v_new, void* out, int32_t* evicted_pos, int32_t* dev_status,
                             void* cuda_stream) {
  vatp_status s = check_params(p, false);
  if (s != VATP_OK) return s;
  const bool windowed = p->indicator == VATP_IND_WINDOW;
  if (!q_new || !k_new || !v_new || !out || !cache_ok(cache, windowed)) return VATP_ERR_INVALID_ARG;
  if (!aligned16(q_new) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out)) return VATP_ERR_INVALID_ARG;
  if (group_of(p) > 1) {
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (p->dtype == VATP_BF16 && p->head_dim == 128 && group_of(p) <= 8) {
      // tensor-core step: the group's heads ride in the rows of the MMA tiles, every K and V row is read once
      Shape sh;
      std::memset(&sh, 0, sizeof(sh));
      sh.units = p->batch * kv_heads_of(p);
      sh.heads = kv_heads_of(p);
      sh.d = p->head_dim;
      sh.scale = p->scale;
      sh.window = windowed ? p->window_w : 0;
      sh.norm = p->norm_kind;
      const cudaError_t e = launch_decode_mma(sh, p->budget, p->n_sink, p->n_recent, *cache, q_new, k_new, v_new, out, evicted_pos,
                                              dev_status, st, (p->flags & VATP_FLAG_DECODE_OVERLAP) != 0, group_of(p));
      if (e != cudaErrorNotSupported) return e == cudaSuccess ? VATP_OK : VATP_ERR_CUDA;
    }
    decode_history_forget(st);
    const cudaError_t e = launch_decode_gqa(p->batch * kv_heads_of(p), group_of(p), p->head_dim, p->dtype, p->budget, p->n_sink,
                                            p->n_recent, windowed ? p->window_w : 0, p->norm_kind, p->scale, *cache, q_new, k_new,
                                            v_new, out, evicted_pos, dev_status, st);
    return e == cudaSuccess ? VATP_OK : (e == cudaErrorNotSupported ? VATP_ERR_UNSUPPORTED : VATP_ERR_CUDA);
  }
  Shape sh;
  std::memset(&sh, 0, sizeof(sh));
  sh.units = p->batch * p->heads;
  sh.heads = p->heads;
  sh.d = p->head_dim;
  sh.scale = p->scale;
  sh.window = windowed ? p->window_w : 0;
  sh.norm = p->norm_kind;
  cudaError_t e = launch_decode(sh, p->dtype, p->budget, p->n_sink, p->n_recent, *cache, q_new, k_new, v_new, out,
                                evicted_pos, dev_status, static_cast<cudaStream_t>(cuda_stream),
                                (p->flags & VATP_FLAG_DECODE_OVERLAP) != 0);
  return e == cudaSuccess ? VATP_OK : VATP_ERR_CUDA;
}

}  // extern "C"
