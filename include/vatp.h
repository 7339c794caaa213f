/*
 * vatp.h - C ABI of the Value-Aware Token Pruning (VATP) hot path for NVIDIA B200 (sm_100a).
 *
 * Method (arXiv 2406.12335, Section 3.2): every cached token k of an attention head has an
 * importance I_k = S_k * ||v_k||_1 (Eq. 4), where S_k is an attention indicator: the attention
 * probability accumulated over all queries so far (Eq. 2, H2O) or over a history window of the
 * last w queries (Eq. 3, Scissorhands).  The lowest-importance tokens are dropped down to a KV
 * budget B; the first F tokens ("Attention Sink Tokens" paragraph) and a local window of the R
 * most recent tokens (Appendix A) are always kept.  Budgets are uniform over heads (Appendix A),
 * so every (batch, head) pair - a "unit" - is an independent problem of identical shape.
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller; the library never allocates,
 *     frees or synchronises.  `params`, `cache` structs are HOST structs read during the call.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = default stream)
 *     and the call returns at once; outputs are valid after the caller synchronises the stream.
 *   - q/k/v are [batch, heads, seq_len, head_dim] with innermost stride 1 and element strides
 *     stride_b / stride_h / stride_t (0 = the contiguous default).  head_dim is 64 or 128.
 *     dtype VATP_BF16 or VATP_F32; all arithmetic accumulates in fp32.
 *   - Data pointers must be 16-byte aligned and row strides multiples of 16 bytes.
 *   - Errors that the host can see (null pointer, bad shape, F + R > B, workspace too small,
 *     misalignment) return a status before anything is launched.  A failed launch returns
 *     VATP_ERR_CUDA.  Device-side conditions (a bounded wait that ran out) are written to
 *     *dev_status (device int32, 0 = fine; caller zeroes it and reads it after sync); the
 *     kernels never trap.
 *   - Grouped-query attention (the Limitations section's "Compatibility with grouped-query
 *     attention", left there to future work with a pointer to a group-wise score): with
 *     params->kv_heads < heads, q (and q_new, out, lse_out) keep `heads` heads while k, v, every
 *     per-token output (attn_acc, vnorm, score, kept_idx) and the decode state have kv_heads heads:
 *     a unit is a (batch, KV head) pair, the G = heads / kv_heads query heads h = g * G .. g * G + G - 1
 *     share KV head g, and the indicator of a cached token is the MEAN over those query heads of its
 *     Eq. 2 / Eq. 3 indicator (prefill), advanced per step by the mean of the heads' probabilities
 *     (decode; with a history window that mean row enters the ring, built after the prefill by
 *     vatp_compact_window, which then needs lse for all `heads` query heads).  Layouts must be
 *     contiguous (stride fields 0); vatp_prefill_scores_from_lse and win_rows (hence vatp_compact
 *     with a history window) are not available with it (VATP_ERR_UNSUPPORTED), and the workspace
 *     holds a normaliser row per query head and G partial indicators.  The decode step takes
 *     the tensor-core kernel for bf16, head_dim 128 and G <= 8 (VATP_FLAG_DECODE_OVERLAP applies as in the multi-head case) and a
 *     general kernel otherwise; the history rebuild runs a general kernel.
 *   - Inputs are assumed finite.
 *   - A second build of the library (compiled with -DVATP_DEBUG_BOUNDS) range-checks every row, slot,
 *     window-row and scratch index its kernels compute before the access; an index outside its array is
 *     not dereferenced, VATP_ERR_BOUNDS goes to *dev_status, and the kernel carries on.  It stands in
 *     for a memory checker where none can be run; results are those of the ordinary build.
 */
#ifndef VATP_H_
#define VATP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  VATP_OK = 0,
  VATP_ERR_INVALID_ARG = 1,
  VATP_ERR_UNSUPPORTED = 2,
  VATP_ERR_WORKSPACE = 3,
  VATP_ERR_CUDA = 4,
  VATP_ERR_TIMEOUT = 5,
  VATP_ERR_STATIC_SCRATCH = 6, /* problem needs more scratch than the built-in array holds */
  VATP_ERR_BOUNDS = 7          /* bounds-checking build only: a kernel computed an index outside its array */
} vatp_status;

typedef enum { VATP_BF16 = 0, VATP_F32 = 1 } vatp_dtype;
typedef enum { VATP_IND_H2O = 0, VATP_IND_WINDOW = 1 } vatp_indicator;
/* Which norm of the value row Eq. 4 multiplies the indicator by.  L1 is the method; L2 and LINF are
 * the variants the Ablation Study compares it with (its table of norms).  The per-slot `vnorm`
 * arrays hold whichever kind the parameters name. */
typedef enum { VATP_NORM_L1 = 0, VATP_NORM_L2 = 1, VATP_NORM_LINF = 2 } vatp_norm_kind;
/* Bits of vatp_params.flags.  VATP_FLAG_DECODE_OVERLAP: see vatp_decode_step. */
typedef enum { VATP_FLAG_DECODE_OVERLAP = 1 } vatp_flags;

/* Problem description shared by the four calls (host struct). */
typedef struct {
  int32_t batch, heads;      /* units = batch * heads                                          */
  int32_t seq_len;           /* T: prompt length (prefill / select / compact)                  */
  int32_t head_dim;          /* d: 64 or 128                                                   */
  int32_t dtype;             /* vatp_dtype of q, k, v, the caches and `out`                    */
  int32_t indicator;         /* vatp_indicator: Eq. 2 or Eq. 3                                 */
  int32_t window_w;          /* w of Eq. 3 (last w queries); ignored for VATP_IND_H2O          */
  float   scale;             /* softmax scale, normally 1/sqrt(d)                              */
  int32_t budget;            /* B: tokens kept per unit                                        */
  int32_t n_sink;            /* F: leading tokens always kept                                  */
  int32_t n_recent;          /* R: most recent tokens always kept; F + R <= B                  */
  int32_t norm_kind;         /* vatp_norm_kind of the value norm in Eq. 4; 0 = the paper's l1   */
  int32_t flags;             /* OR of vatp_flags; 0 = none                                     */
  int32_t kv_heads;          /* grouped-query attention: KV heads (a divisor of heads); 0 or
                                == heads = multi-head attention.  See "Grouped-query attention" */
  int64_t stride_b, stride_h, stride_t; /* element strides of q, k, v; 0 = contiguous          */
} vatp_params;

/*
 * Decode-time state of all units (host struct of caller-owned DEVICE arrays).
 * cap = vatp_cache_capacity(budget) slots per unit: budget + 1 rounded up to a multiple of 8 (one
 * slot beyond the budget receives the incoming token before the eviction; the padding keeps every
 * unit's arrays 32-byte aligned).  Slot order is not positional after evictions; pos[] gives each
 * slot's original token position (-1 = empty slot).  acc, vnorm and pos must be 16-byte aligned.
 */
typedef struct {
  void    *k_cache, *v_cache; /* [batch, heads, cap, head_dim], params dtype                   */
  float   *acc;               /* [batch, heads, cap] indicator S per slot (Eq. 2 / Eq. 3)      */
  float   *vnorm;             /* [batch, heads, cap] ||v||_1 per slot (Eq. 4)                  */
  int32_t *pos;               /* [batch, heads, cap] original position per slot, -1 = empty    */
  int32_t *len;               /* [batch, heads] live tokens                                    */
  int32_t *free_slot;         /* [batch, heads] slot the next token is written to              */
  int32_t *next_pos;          /* [batch, heads] position t of the next token                   */
  float   *ring;              /* windowed only: [batch, heads, w, cap] last w probability rows,
                                 row (j mod w) holds query position j; else NULL                */
  int64_t *acc_fixed;         /* windowed only: [batch, heads, cap] exact fixed-point window sum */
  int32_t *last_slot;         /* [batch, heads] slot the previous step wrote its token to, -1 after
                                 compaction; lets a step that overlaps the tail of the previous one
                                 re-read that one row                                            */
} vatp_cache;

/* Slots per unit of the decode state for a budget of B tokens (see vatp_cache). */
int32_t vatp_cache_capacity(int32_t budget);

/* Bytes of device scratch that vatp_prefill_scores / vatp_select need for `params`. */
size_t vatp_workspace_bytes(const vatp_params* params);

/*
 * Prefill scoring (Eq. 1-4 at t = T-1), without materialising the T x T matrix.
 *   pass 1: lse[j] = log sum_{i<=j} exp(scale * <q_j, k_i>)           (row normaliser of Eq. 1)
 *   pass 2: attn_acc[k] = sum_j exp(scale * <q_j, k_k> - lse[j]) over j >= k (Eq. 2), or over
 *           j >= max(T - w, k) (Eq. 3, last w queries); QK^T is recomputed, never stored
 *   vnorm[k] = sum_c |v[k][c]|,  score[k] = attn_acc[k] * vnorm[k]     (Eq. 4)
 * q, k, v: inputs as described above (read only).
 * lse_out:  [batch, heads, T] fp32 output (natural log), nullable.
 * attn_acc, vnorm, score: [batch, heads, T] fp32 outputs.
 * win_rows: VATP_IND_WINDOW only, nullable: [batch, heads, w, T] fp32 output, row r = probabilities
 *           of query T - w + r (zero where masked or where T - w + r < 0), for vatp_compact.  NULL
 *           (always for H2O): nothing is written per (query, key) pair; the decode state of the
 *           history window is then built by vatp_compact_window, which recomputes the kept columns.
 * workspace: >= vatp_workspace_bytes(params) bytes of device scratch, 256-byte aligned; holds the
 *           row normalisers between the two passes and two work-item counters.
 * bf16 with head_dim 128 runs on the tensor cores; other combinations use an fp32 FMA kernel.
 */
vatp_status vatp_prefill_scores(const vatp_params* params, const void* q, const void* k, const void* v,
                                float* lse_out, float* attn_acc, float* vnorm, float* score,
                                float* win_rows, void* workspace, size_t workspace_bytes,
                                int32_t* dev_status, void* cuda_stream);

/*
 * Prefill scoring when the row normalisers of Eq. 1 already exist.  The Limitations section
 * ("FlashAttention Support for H2O") names the cost this removes: a fused attention kernel does not
 * return the attention matrix, so accumulated attention (Eq. 2) seemed to need the O(n^2) matrix.
 * Such a kernel does return, per query row j, lse[j] = log sum_{i<=j} exp(scale * <q_j, k_i>);
 * given those, pass 1 above is skipped and the indicator costs ONE recomputation of QK^T:
 *   attn_acc[k] = sum_j exp(scale * <q_j, k_k> - lse_in[j])   (Eq. 2, or Eq. 3 over the last w rows)
 *   vnorm, score as in vatp_prefill_scores (Eq. 4).
 * lse_in:  [batch, heads, T] fp32 device array, natural log, 16-byte aligned, read only; it must
 *          be the causal row normaliser for the same q, k and scale (the result is as accurate as
 *          lse_in is: an error e in lse_in[j] scales row j's probabilities by exp(-e)).  With
 *          VATP_IND_WINDOW only rows j >= T - w are read.
 * lse_out: nullable; receives a copy of lse_in.  All other arguments, the workspace requirement
 *          and the error behaviour are those of vatp_prefill_scores; NULL lse_in is
 *          VATP_ERR_INVALID_ARG.
 */
vatp_status vatp_prefill_scores_from_lse(const vatp_params* params, const void* q, const void* k, const void* v,
                                         const float* lse_in, float* lse_out, float* attn_acc, float* vnorm,
                                         float* score, float* win_rows, void* workspace, size_t workspace_bytes,
                                         int32_t* dev_status, void* cuda_stream);

/*
 * Attention forward fused with prefill scoring: the layer's output rows (Section 3.1, Eq. 1)
 *   attn_out[j] = sum_{i<=j} a_i^j v_i
 * and the row normalisers come out of ONE streaming sweep over K and V (never materialising the
 * T x T matrix), and the indicator then costs one recomputation of QK^T (pass 2 of
 * vatp_prefill_scores).  A caller that needs the attention output anyway - every prefill does -
 * pays three contraction sweeps for output, indicator and importance together instead of the
 * forward's two plus the scoring call's two: the remedy for the cost the Limitations section names
 * ("FlashAttention Support for H2O"), built in.
 * attn_out: [batch, heads, T, head_dim] contiguous device array of the params dtype, 16-byte
 *           aligned, output; required (NULL is VATP_ERR_INVALID_ARG).  bf16 carries the rounding
 *           of the probabilities to bf16 before they meet V (as fused attention kernels do):
 *           |error| <= 2^-8 * max|v| per element, typically far less.
 * All other arguments, outputs, the workspace requirement and the error behaviour are those of
 * vatp_prefill_scores; both indicators (Eq. 2, Eq. 3) and grouped-query attention (one forward per
 * query head of the KV groups, attn_out covering all `heads` query heads) are supported; head_dim > 256
 * outside the tensor-core shape is not (VATP_ERR_UNSUPPORTED).
 */
vatp_status vatp_prefill_attention_scores(const vatp_params* params, const void* q, const void* k, const void* v,
                                          void* attn_out, float* lse_out, float* attn_acc, float* vnorm, float* score,
                                          float* win_rows, void* workspace, size_t workspace_bytes,
                                          int32_t* dev_status, void* cuda_stream);

/*
 * vatp_prefill_scores for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is a packaging variant of the call above and computes exactly the same thing.)
 *
 * Who needs it: code that runs where cudaMalloc is not an option - a plugin inside a host
 * application that owns all device memory and offers no scratch, a real-time loop that must never
 * hit the device-wide synchronisation an allocation implies, or a process whose pool was sized up
 * front.  Such callers still own q, k, v and the outputs, but have nowhere to put the row
 * normalisers that pass 1 hands to pass 2.  Here that scratch is a fixed device array built into
 * the library: VATP_STATIC_SCRATCH_BYTES on every GPU that loads the library, held until the
 * process exits.  The call allocates and frees nothing.
 *
 * Arguments are those of vatp_prefill_scores without workspace / workspace_bytes.
 * Limit: vatp_workspace_bytes(params) <= VATP_STATIC_SCRATCH_BYTES, i.e. batch * heads *
 * round_up(seq_len, 256) <= 1,048,576 (for example 32 heads x 32768 tokens, or 256 units x 4096);
 * anything larger returns VATP_ERR_STATIC_SCRATCH before a launch.
 * First call on a device: looks up the array's device address (once per device, with the current
 * device) - make that first call outside any stream capture.
 * Sharing: all calls on a device use the same array.  Calls on one stream are ordered and safe
 * (each call starts by zeroing its counters - a memset, or a kernel that first waits for all
 * earlier work in the stream - and touches nothing else before that, so it cannot begin before
 * the previous call on the stream has finished with the array);
 * calls that may overlap on the GPU (different streams, different host threads) race on it and
 * give wrong scores - serialise them, or use vatp_prefill_scores with separate workspaces.  The
 * array keeps the previous call's contents; nothing in it needs clearing, because pass 1 writes
 * every normaliser that pass 2 reads.
 */
#define VATP_STATIC_SCRATCH_BYTES ((4u << 20) + 256u)
vatp_status vatp_prefill_scores_static(const vatp_params* params, const void* q, const void* k, const void* v,
                                       float* lse_out, float* attn_acc, float* vnorm, float* score,
                                       float* win_rows, int32_t* dev_status, void* cuda_stream);

/*
 * Budgeted selection (Section 3.2 with Appendix A's budget split): per unit keep the first F
 * tokens, the last R tokens and the B - F - R highest-`score` tokens of the range [F, T - R);
 * among equal scores the lower index is kept.  T <= B keeps every token.
 * score: [batch, heads, T] fp32 (non-negative).
 * kept_idx: [batch, heads, B] int32 output, ascending; when T < B entries T..B-1 are -1.
 */
vatp_status vatp_select(const vatp_params* params, const float* score, int32_t* kept_idx,
                        void* workspace, size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * Compaction: gather the surviving K/V rows (bit-exact copies, ascending original index) into
 * the budgeted cache and initialise the decode state: acc <- attn_acc[kept], vnorm <- vnorm[kept],
 * pos <- kept index, len <- min(T, B), free_slot <- len, next_pos <- T, last_slot <- -1; unused slots
 * get pos -1.
 * VATP_IND_WINDOW also gathers win_rows columns into `ring` (row (T - w + r) mod w) and sets
 * acc_fixed to the fixed-point window sums; win_rows is then required (see vatp_compact_window for
 * the variant that needs none).
 */
vatp_status vatp_compact(const vatp_params* params, const void* k, const void* v, const float* attn_acc,
                         const float* vnorm, const float* win_rows, const int32_t* kept_idx,
                         const vatp_cache* cache, int32_t* dev_status, void* cuda_stream);

/*
 * Compaction for the history-window indicator (Eq. 3) without the [w, T] probability rows.  The
 * Limitations section notes that this indicator only needs the attention of the last w queries;
 * of those w x T probabilities the decode state keeps the B kept columns.  This call gathers K/V and
 * initialises the state as vatp_compact does, and recomputes the kept block itself:
 *   ring[(j mod w)][slot] = exp(scale * <q_j, k_slot> - lse[j]) for T - w <= j < T, pos[slot] <= j
 *   acc_fixed[slot] = sum over those j of the 2^52 fixed-point image, acc[slot] = that sum as float
 * (a w x B x d contraction per unit), so vatp_prefill_scores may be called with win_rows = NULL.
 * q: the prompt's queries (as given to vatp_prefill_scores); lse: [batch, heads, T] fp32 natural-log
 * row normalisers (lse_out of vatp_prefill_scores, or an attention forward's), of which rows
 * j >= T - w are read.  Other arguments and errors as vatp_compact; params->indicator must be
 * VATP_IND_WINDOW.  The recomputed probabilities equal those of the scoring pass to fp32 rounding,
 * not bit for bit (another kernel sums the dot products in another order).
 */
vatp_status vatp_compact_window(const vatp_params* params, const void* q, const void* k, const void* v,
                                const float* lse, const float* attn_acc, const float* vnorm,
                                const int32_t* kept_idx, const vatp_cache* cache, int32_t* dev_status,
                                void* cuda_stream);

/*
 * One generation step on the budgeted cache (Eq. 1-4 at step t = next_pos):
 *   write (k_new, v_new) into free_slot with pos = t; p = softmax(scale * <q_new, k_i>) over all
 *   live slots (the new token included); out = sum_i p_i v_i (Eq. 1); acc_i += p_i (Eq. 2; the
 *   new token starts at its own probability) or the window update of Eq. 3; then, if more than
 *   B tokens are live, the slot with the smallest acc_i * vnorm_i among tokens with
 *   F <= pos <= t - R is released (ties: the highest position goes).
 * q_new, k_new, v_new: [batch, heads, head_dim]; out: same shape and dtype.
 * evicted_pos: [batch, heads] int32, nullable; position released this step or -1.
 * State arrays are updated in place.  seq_len in params is ignored.
 *
 * Ordering on the stream.  The step is enqueued as a launch that may begin while the work before it
 * in the stream is still draining.  By default that is invisible: before anything else, the step only
 * requests K/V cache tiles; it reads q_new, k_new, v_new and the state, and writes anything, only after
 * all earlier work in the stream has completed, and it re-reads the one cache row the previous step
 * appended.  The only assumption is about those early tile reads: between the compaction (or the
 * previous step) and this step, cache rows are written by calls of this library only, or by kernels of
 * the caller that do not release their dependents before they finish (ordinary launches do not).
 *
 * VATP_FLAG_DECODE_OVERLAP in params->flags opts in to more.  The library then keeps, per stream, the
 * buffers of its recent decode launches; a step whose buffers (cache arrays, q_new, k_new, v_new, out,
 * evicted_pos) overlap none of the launches that can still be running starts reading at once and runs
 * beside them - steps of different layers' or sequences' caches issued back to back.  Steps that share a
 * buffer with such a launch behave as in the default.  The caller then guarantees that every input of a
 * flagged step was complete in memory before the previous vatp_decode_step on the stream was enqueued,
 * or was written by an earlier vatp_decode_step; put differently: after enqueueing other work that
 * produces a step's inputs, make the first step call without the flag.  Any other call of this library
 * on the stream (prefill, selection, compaction) ends the record by itself.  Under stream capture the
 * record is kept per capture, and the first step recorded into a graph always waits, so a replay is
 * valid whatever ran before it.
 */
vatp_status vatp_decode_step(const vatp_params* params, const vatp_cache* cache, const void* q_new,
                             const void* k_new, const void* v_new, void* out, int32_t* evicted_pos,
                             int32_t* dev_status, void* cuda_stream);

/*
 * Self-test of the bounded device-side waits (every pipeline wait in this library gives up after a
 * time limit, writes VATP_ERR_TIMEOUT to *dev_status and lets the kernel return; nothing traps).
 * Launches one CTA that waits on a barrier nobody arms for `limit_ns` nanoseconds (1 .. 1e8).
 * dev_status: device int32, set to VATP_ERR_TIMEOUT by the kernel; waited_ns: device uint64,
 * nullable, receives the time actually waited.  The paper has no counterpart.
 */
vatp_status vatp_selftest_bounded_wait(uint64_t limit_ns, int32_t* dev_status, uint64_t* waited_ns, void* cuda_stream);

/*
 * Host-only probe of the rule that lets consecutive vatp_decode_step launches overlap on the GPU (no
 * device work, usable without a GPU).  Pretends that a launch on `stream` reads and writes the n
 * (<= 13) host-described byte ranges [begin[i], begin[i] + bytes[i]) and keeps `share` of the
 * machine's CTA slots until the launch before it has completed.  Returns 1 when that launch would
 * run without waiting for its predecessors - it overlaps none of the recorded launches that can
 * still be resident - else 0, and records it; -1 on bad arguments.  A negative `share` instead ends
 * the stream's record, as every other call of this library on a stream does (the next launch then
 * waits), and returns 0.  `stream` is only a key (use values no real stream has).  The launches
 * probed here count as having opted in (VATP_FLAG_DECODE_OVERLAP).  The paper has no counterpart.
 */
int32_t vatp_selftest_overlap_policy(void* stream, const uint64_t* begin, const uint64_t* bytes, int32_t n, double share);

const char* vatp_status_string(vatp_status status);

#ifdef __cplusplus
}
#endif
#endif /* VATP_H_ */
