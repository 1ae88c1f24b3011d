/*
 * daf.h - C ABI of the B200 (sm_100a) library for the prefill-attention path of
 * Decoupled Attention Fusion (DAF).
 *
 * The path, per layer (paper, section "Methods", items 1-3):
 *   daf_select          important-token selection, gather into the condensed
 *                       sequence, hybrid KV-cache update              (items 1, 2)
 *   daf_important_attn  self-attention among the condensed tokens     (item 1)
 *   daf_qd_attn         question rows over the hybrid cache           (item 2)
 *   daf_imp_qd_attn     the two attention stages from one list of work items (items 1, 2)
 *   daf_fuse            state fusion into the final hidden-state rows (item 3)
 *   daf_full_causal_attn  full recomputation, the comparison path (section
 *                       "Preliminary Results", the full-recompute baseline)
 *
 * Conventions, unless an argument says otherwise
 *   - Every data pointer is a DEVICE pointer owned by the caller, 16-byte
 *     aligned.  The library allocates no device memory; scratch comes from the
 *     caller's `workspace` (size from daf_workspace_bytes), which must not be
 *     shared by calls that may overlap on the GPU.
 *   - Tensors are token-major [tokens, heads, head_dim], bf16, contiguous,
 *     head_dim = 128.  N = L_d + L_q.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*, NULL = the
 *     default stream) and return without synchronising.
 *   - Return value: DAF_OK or a negative daf_status.  Arguments are validated on
 *     the host before anything is launched; a call that fails validation
 *     launches nothing.  Device-side problems (a bounded wait that ran out)
 *     are recorded in the workspace status word and read by daf_poll_status.
 *     Nothing aborts, traps or throws.
 */
#ifndef DAF_H_
#define DAF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum daf_status {
    DAF_OK = 0,
    DAF_ERR_INVALID_ARG = -1, /* NULL where a buffer is required, negative size, r out of range, ... */
    DAF_ERR_UNSUPPORTED = -2, /* head_dim != 128, n_q_heads % n_kv_heads != 0, sizes beyond the limits  */
    DAF_ERR_ALIGNMENT = -3,   /* a pointer or a row stride is not a multiple of 16 bytes              */
    DAF_ERR_WORKSPACE = -4,   /* workspace missing or smaller than daf_workspace_bytes                */
    DAF_ERR_CUDA = -5,        /* a CUDA runtime/driver call failed; see daf_last_cuda_error           */
    DAF_ERR_TIMEOUT = -6,     /* device: a bounded barrier wait ran out (from daf_poll_status)        */
    DAF_ERR_BOUNDS = -7       /* device: an index outside its tensor was skipped (from daf_poll_status) */
} daf_status;

/* Problem statement of one layer (paper, "Methods", notation paragraph: L_d, L_q, r). */
typedef struct daf_params {
    int32_t L_d;              /* total document tokens                                   */
    int32_t L_q;              /* question tokens (may be 0)                              */
    double  r;                /* fraction of document tokens recomputed, 0 <= r <= 1     */
    int32_t n_q_heads;        /* query heads                                              */
    int32_t n_kv_heads;       /* key/value heads; must divide n_q_heads                   */
    int32_t head_dim;         /* must be 128                                              */
    float   softmax_scale;    /* <= 0 selects 1/sqrt(head_dim)                            */
    int32_t fuse_mode;        /* 0: compact rows [important ; question]  1: scatter to original positions */
    int32_t overwrite_doc_kv; /* 1 (the paper's hybrid cache): important rows of the document cache are
                                 replaced by fresh K/V.  0: document rows stay offline (ablation).       */
} daf_params;

/* Number of important tokens k = ceil(r * L_d), clamped to [0, L_d].  r*L_d is
 * shrunk by a relative 1e-6 first so that an r rounded to single precision gives
 * the intended count.  (Methods, notation paragraph: r, the share of the document tokens that is recomputed.) */
int32_t daf_num_important(int32_t L_d, double r);

/* Bytes of device scratch every call below may need for this problem (selection
 * keys and histograms, split-KV partial results, the status word). */
size_t daf_workspace_bytes(const daf_params* p);

/* Clears the status word at the head of a freshly allocated workspace.  Call once
 * per workspace before its first use (a workspace that is all zero bytes needs no call). */
int daf_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Comparison variant, not part of the DAF path (Complexity Analysis paragraph: selective recomputation
 * in which the important rows and the question rows attend the FULL context costs about
 * r L_d^2 + L_d L_q, against r^2 L_d^2 + L_q (L_d + L_q) for DAF).  Same kernel, with a position per row:
 *   q_rows   [n_rows, n_q_heads, 128] compact query rows (important rows in position order, then question rows)
 *   kv_k, kv_v  [N, n_kv_heads, 128]  the hybrid cache
 *   row_pos  int32 [n_rows] ascending original positions (as daf_fuse / daf_layer report in row_pos_out);
 *            row j attends keys t <= row_pos[j]
 *   out      bf16 rows j at out + j * out_row_stride_bytes; lse optional fp32 [n_q_heads, n_rows]
 */
int daf_blend_attn(const daf_params* p, int32_t n_rows, const void* q_rows, const void* kv_k, const void* kv_v,
                   const int32_t* row_pos, void* out, int64_t out_row_stride_bytes, float* lse,
                   void* workspace, size_t workspace_bytes, void* stream);

/* Per-layer importance signal (Methods item 1: tokens are ranked by the deviation between the
 * fresh and the offline KV states of a layer; signals of several layers are then aggregated by
 * daf_select).  The paper gives no formula; this library takes, for document token i,
 *     s[i] = sum over heads and channels of (Kf - Kc)^2 + (Vf - Vc)^2      (fp32 accumulation).
 *   k_fresh, v_fresh    [>= L_d, n_kv_heads, 128] fresh K/V of one layer (rows >= L_d are ignored)
 *   k_cached, v_cached  [>= L_d, n_kv_heads, 128] offline K/V of the same layer
 *   scores_row          fp32 [L_d] out: one row of the [n_sig, L_d] matrix daf_select takes
 */
int daf_deviation_scores(const daf_params* p, const void* k_fresh, const void* v_fresh, const void* k_cached,
                         const void* v_cached, float* scores_row, void* stream);

/* Step 1 (Methods item 1 "selection", "gather"; item 2 "hybrid KV cache").
 *   scores   fp32 [n_sig, L_d] per-layer importance signals, summed over n_sig in
 *            ascending row order in fp32; the k highest sums are selected (ties:
 *            lower position first; NaN ranks lowest).  NULL: use idx_in instead.
 *   idx_in   int32 [k] strictly increasing positions in [0, L_d); read iff scores == NULL.
 *   q_fresh  [N, n_q_heads, 128]; k_fresh, v_fresh [N, n_kv_heads, 128]   (read only)
 *   kv_k, kv_v  [N, n_kv_heads, 128] IN/OUT: rows < L_d hold the offline document
 *            cache on entry.  On exit rows idx hold fresh K/V (if overwrite_doc_kv)
 *            and rows L_d..N-1 hold the fresh question K/V.  Must not alias k_fresh/v_fresh.
 *   idx_out  int32 [k] selected positions, ascending (also written when idx_in is given)
 *   q_pack   [k, n_q_heads, 128]; k_pack, v_pack [k, n_kv_heads, 128]: rows idx of the fresh tensors.
 *            q_pack may be NULL when no packed copy of the Q rows is wanted (daf_layer and
 *            daf_imp_qd_attn can read them in place).  k_pack and v_pack may be NULL, both or
 *            neither, when no packed copies of the K/V rows are wanted (daf_layer can read them
 *            in place); the cache update is done all the same.
 */
int daf_select(const daf_params* p, const float* scores, int32_t n_sig, const int32_t* idx_in,
               const void* q_fresh, const void* k_fresh, const void* v_fresh,
               void* kv_k, void* kv_v,
               int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack,
               void* workspace, size_t workspace_bytes, void* stream);

/* The selection of step 1 alone: aggregates the score rows and writes the k selected positions, ascending, to
 * idx_out; nothing is gathered.  For callers that schedule the selection apart from the rest of the layer -- it
 * depends only on the scores, so it can run on another stream while an earlier layer's attention is still under
 * way -- and then pass the positions to daf_select or daf_layer as idx_in.  Same result as daf_select's idx_out. */
int daf_select_topk(const daf_params* p, const float* scores, int32_t n_sig, int32_t* idx_out,
                    void* workspace, size_t workspace_bytes, void* stream);

/* Step 1 starting from K/V instead of from scores (Methods item 1: the deviation signals of several layers,
 * typically the 2nd to 4th, are aggregated and the tokens ranked by the aggregate).  The signal of layer l is
 * the one daf_deviation_scores computes; the layers are added in ascending order in fp32, exactly as daf_select
 * adds the rows of a score matrix, and the k highest sums are selected.  The per-layer score matrix is never
 * written: one kernel streams the signal layers' K/V once and leaves one fp32 sum per document token.
 *   n_sig           number of signal layers, 1..8
 *   sig_k_fresh, sig_v_fresh, sig_k_cached, sig_v_cached
 *                   HOST arrays of n_sig DEVICE pointers: fresh and offline K/V of each signal layer,
 *                   [>= L_d, n_kv_heads, 128] each (the arrays are read before the call returns)
 *   q_fresh ... v_pack   the layer being processed, exactly as in daf_select (gather and cache update)
 *   signal_sum_out  optional fp32 [L_d] (device): receives the aggregated signal; NULL keeps it in the workspace
 */
int daf_select_from_kv(const daf_params* p, int32_t n_sig, const void* const* sig_k_fresh, const void* const* sig_v_fresh,
                       const void* const* sig_k_cached, const void* const* sig_v_cached,
                       const void* q_fresh, const void* k_fresh, const void* v_fresh, void* kv_k, void* kv_v,
                       int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack, float* signal_sum_out,
                       void* workspace, size_t workspace_bytes, void* stream);

/* Step 2 (Methods item 1; the r^2 L_d^2 term of the complexity analysis): causal
 * softmax attention among the k packed rows, query head h reading KV head
 * h / (n_q_heads / n_kv_heads).  bf16 operands, fp32 accumulation and softmax.
 *   out      bf16; packed row j, head h goes to
 *            out + dst_rows[j] * out_row_stride_bytes + h * 256   (dst_rows == NULL: row j)
 *   lse      optional fp32 [n_q_heads, k]: natural-log sum of exponentials of each row
 */
int daf_important_attn(const daf_params* p, int32_t k,
                       const void* q_pack, const void* k_pack, const void* v_pack,
                       void* out, int64_t out_row_stride_bytes, const int32_t* dst_rows, float* lse,
                       void* workspace, size_t workspace_bytes, void* stream);

/* Step 3 (Methods item 2): the L_q question rows attend over the L_d + L_q rows of
 * the hybrid cache; question row i sits at position L_d + i and sees keys <= L_d + i.
 *   q_question  [L_q, n_q_heads, 128]  (= q_fresh + L_d rows)
 *   kv_k, kv_v  [N, n_kv_heads, 128]   the hybrid cache left by daf_select
 *   out, out_row_stride_bytes, dst_rows, lse: as in daf_important_attn, with L_q rows
 */
int daf_qd_attn(const daf_params* p, const void* q_question, const void* kv_k, const void* kv_v,
                void* out, int64_t out_row_stride_bytes, const int32_t* dst_rows, float* lse,
                void* workspace, size_t workspace_bytes, void* stream);

/* Steps 2 and 3 together, the way daf_layer runs them: one attention launch over the work
 * items of both stages (long causal chains of step 2 and the KV axis of step 3 are cut into
 * ranges) and one launch that merges the ranges' partial results.  Results equal those of
 * daf_important_attn + daf_qd_attn up to fp32 summation order.  State fusion (Methods item 3)
 * is done by the epilogues as in daf_layer:
 *   q_pack, k_pack, v_pack   the k packed rows left by daf_select.  q_pack may be NULL: the Q row of
 *            packed row j is then read in place, row idx[j] of q_fresh ([>= L_d, n_q_heads, 128]),
 *            which saves writing and re-reading the largest of the packed tensors but costs every
 *            work item a scattered fetch; measured on B200 the layer time changes by -2 % at
 *            k = 41780, +-1 % at k = 6554 and +10 % at k = 922.
 *   q_question, kv_k, kv_v   as in daf_qd_attn
 *   idx      int32 [k] positions of the packed rows; read iff p->fuse_mode == 1 or q_pack == NULL
 *   hidden   bf16, row stride n_q_heads * 256 bytes.  fuse_mode 0: rows 0..k-1 are the
 *            important rows in position order, rows k..k+L_q-1 the question rows;
 *            fuse_mode 1: [N rows], important row j at row idx[j], question row i at row L_d + i,
 *            other rows untouched.
 * Both k and L_q must be positive (use the single-stage calls otherwise). */
int daf_imp_qd_attn(const daf_params* p, const void* q_pack, const void* q_fresh, const void* k_pack, const void* v_pack,
                    const void* q_question, const void* kv_k, const void* kv_v, const int32_t* idx,
                    void* hidden, void* workspace, size_t workspace_bytes, void* stream);

/* Measurement aid (no counterpart in the paper): daf_imp_qd_attn with only part of its work enqueued, so
 * that the attention launch and the merge launch can be timed apart.  launches = 1: the attention launch
 * alone (final rows of the items that cover all their keys, partial results of the others, into the
 * workspace); 2: the merge launch alone (reads the partial results a launches = 1 call left in the same
 * workspace); 3: both, i.e. daf_imp_qd_attn.  Other values: DAF_ERR_INVALID_ARG. */
int daf_imp_qd_attn_launches(const daf_params* p, const void* q_pack, const void* q_fresh, const void* k_pack,
                             const void* v_pack, const void* q_question, const void* kv_k, const void* kv_v,
                             const int32_t* idx, void* hidden, void* workspace, size_t workspace_bytes, void* stream,
                             int32_t launches);

/* daf_qd_attn for callers that cannot provide a workspace.  (The paper has no
 * counterpart of this entry point; it exists for integration only.)
 *
 * Who needs it: code that runs where device memory can no longer be obtained,
 * e.g. inside a serving process whose memory pool already owns the whole GPU,
 * or inside another framework's allocator scope where a driver allocation would
 * stall every stream.  Such a caller passes inputs and outputs only; the status
 * word and the split-KV partial results of the question-document stage live in
 * a fixed 16 MiB array that is part of this library's device image (each GPU
 * that loads the library holds it until the process exits).  The call makes no
 * cudaMalloc/cudaFree and calls no allocating routine.
 *
 *   - Arguments as in daf_qd_attn, without workspace.
 *   - Problems whose scratch need exceeds daf_qd_attn_static_max_bytes() are
 *     rejected with DAF_ERR_WORKSPACE before anything is launched.
 *   - The first call on each device looks up the array's device address (with
 *     that device current); make that first call outside any stream capture.
 *   - All calls on one device share the array, and it keeps the previous call's
 *     contents; the call clears the part that must start at zero.  Two calls that
 *     may overlap on the GPU (different streams) race on it: serialise them.
 *   - Device-side status (a bounded wait that ran out) is kept at the head of
 *     that array: daf_qd_attn_static_poll_status reads and clears it, as
 *     daf_poll_status does for a workspace, also without allocating.
 *   - Host threads may make their first calls concurrently; they resolve the same
 *     address.  Results are exactly those of daf_qd_attn. */
int daf_qd_attn_static(const daf_params* p, const void* q_question, const void* kv_k, const void* kv_v,
                       void* out, int64_t out_row_stride_bytes, const int32_t* dst_rows, float* lse,
                       void* stream);
size_t daf_qd_attn_static_max_bytes(void);
int daf_qd_attn_static_poll_status(void* stream);

/* Step 4 (Methods item 3), stand-alone form: copy o_imp [k, n_q_heads*128] and
 * o_q [L_q, n_q_heads*128] into `hidden`: compact mode -> rows 0..k+L_q-1 of a
 * [k+L_q, n_q_heads*128] buffer; scatter mode -> rows idx and L_d..N-1 of an
 * [N, n_q_heads*128] buffer (other rows untouched).  row_pos_out (optional, int32
 * [k+L_q]) receives the original position of each compact row.  The two attention
 * calls can write these rows themselves through out/dst_rows; this call exists for
 * callers that keep the stage outputs separate. */
int daf_fuse(const daf_params* p, int32_t k, const int32_t* idx, const void* o_imp, const void* o_q,
             void* hidden, int32_t* row_pos_out, void* stream);

/* Comparison path: causal attention over n_tokens fresh rows (full recomputation). */
int daf_full_causal_attn(const daf_params* p, int32_t n_tokens, const void* q, const void* k, const void* v,
                         void* out, float* lse, void* workspace, size_t workspace_bytes, void* stream);

/* One whole layer, steps 1-4 in order with the fusion done by the attention
 * epilogues (device pointers; arguments as in daf_select, plus)
 *   hidden       compact: [k+L_q, n_q_heads*128]; scatter: [N, n_q_heads*128]
 *   row_pos_out  optional int32 [k+L_q]
 *   q_pack       may be NULL when L_q > 0: step 2 then reads its Q rows in place (see daf_imp_qd_attn)
 *   k_pack, v_pack  may be NULL (both or neither) when k > 0 and L_q > 0: step 2 then reads its K/V rows in
 *                place too -- rows idx of k_fresh / v_fresh, fetched by the attention kernel itself -- and
 *                the kernel in front of it only updates the hybrid cache.  Same results, bit for bit, and no
 *                packed buffers to provide; measured slower than the packed form at every size tried (the
 *                rows are re-read by every query tile of their KV group), so pass the buffers where time matters.
 *                DAF_ERR_INVALID_ARG if only one of the two is NULL, or if they are NULL while L_q == 0.
 */
int daf_layer(const daf_params* p, const float* scores, int32_t n_sig, const int32_t* idx_in,
              const void* q_fresh, const void* k_fresh, const void* v_fresh, void* kv_k, void* kv_v,
              int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack,
              void* hidden, int32_t* row_pos_out,
              void* workspace, size_t workspace_bytes, void* stream);

/* Offline cache stored in fp8 (no counterpart in the paper beyond its remark, under Limitations, that storing the
 * offline KV caches is the bottleneck at scale).  The document rows of a layer's offline cache are kept as one byte per
 * element in the 8-bit floating-point format with 1 sign, 4 exponent (bias 7) and 3 mantissa bits (no infinities,
 * S.1111.111 = NaN), with one fp32 scale per KV head; only the layer being processed is expanded to bf16:
 *     kv[t, h, d] = bf16( scale[h] * value(byte[t, h, d]) )      fp32 product, both roundings to nearest-even
 * into rows [0, L_d) of the hybrid-cache buffer, after which the path is the bf16 path: the important rows are
 * overwritten with fresh bf16 K/V and the question rows appended, exactly as in daf_select.  The fp8 cache itself
 * is read-only, so a resident offline cache costs half the bytes and one [N, n_kv_heads, 128] bf16 buffer pair is
 * reused from layer to layer.
 *   k_cached_fp8, v_cached_fp8  [L_d, n_kv_heads, 128] bytes (device)
 *   k_scale, v_scale            fp32 [n_kv_heads] (device), or NULL for 1
 *   kv_k, kv_v                  [N, n_kv_heads, 128] bf16 OUT
 * daf_layer_fp8 = this expansion followed by daf_layer (same remaining arguments); the selection kernel runs
 * beside the expansion, which it does not depend on. */
int daf_expand_fp8_cache(const daf_params* p, const void* k_cached_fp8, const void* v_cached_fp8, const float* k_scale,
                         const float* v_scale, void* kv_k, void* kv_v, void* stream);
int daf_layer_fp8(const daf_params* p, const float* scores, int32_t n_sig, const int32_t* idx_in,
                  const void* q_fresh, const void* k_fresh, const void* v_fresh,
                  const void* k_cached_fp8, const void* v_cached_fp8, const float* k_scale, const float* v_scale,
                  void* kv_k, void* kv_v, int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack,
                  void* hidden, int32_t* row_pos_out, void* workspace, size_t workspace_bytes, void* stream);

/* The same layer for callers whose tensors live in HOST memory (pinned memory
 * makes the copies asynchronous).  h_* are host pointers; every copy to and from
 * the device is part of the call.  `arena` is caller-owned device memory of at
 * least daf_layer_host_arena_bytes(p) bytes.
 *   h_kv_k, h_kv_v  [N, n_kv_heads, 128] host IN/OUT like kv_k/kv_v above
 *                   (copied back only if copy_back_kv != 0)
 *   h_hidden        host output, layout by fuse_mode (compact mode recommended)
 *   h_idx_out       host int32 [k] (optional)
 * The call synchronises `stream` before returning.
 * Of the fresh tensors a layer touches only the rows of the important tokens and of the question: when h_q_fresh,
 * h_k_fresh and h_v_fresh are all pinned memory that the device can address, those rows are read straight from the
 * host by the gather / cache-update kernel (k + L_q rows cross the link instead of N) and only the question's Q rows
 * are copied; otherwise the three tensors are copied whole.  Same results either way.
 *
 * daf_layer_host_begin / daf_layer_host_end are the two halves of that call: `begin` (same arguments) enqueues the
 * copies in, the layer and the copies out on `stream` and returns without waiting; `end` waits for `stream` and
 * returns the layer's status.  A caller with two arenas and two streams begins layer i + 1 before it ends layer
 * i, so that the copies in of one layer run beside the kernels and the copies out of the other (the link to the
 * host carries both directions at once).  Between `begin` and `end` the host buffers and the arena belong to the
 * call; the host buffers must be pinned for the copies to overlap anything.  `end` without a `begin` on that
 * arena returns whatever status word the arena holds. */
size_t daf_layer_host_arena_bytes(const daf_params* p);
int daf_layer_host(const daf_params* p, const float* h_scores, int32_t n_sig, const int32_t* h_idx_in,
                   const void* h_q_fresh, const void* h_k_fresh, const void* h_v_fresh,
                   void* h_kv_k, void* h_kv_v, int32_t copy_back_kv,
                   void* h_hidden, int32_t* h_idx_out,
                   void* arena, size_t arena_bytes, void* stream);
int daf_layer_host_begin(const daf_params* p, const float* h_scores, int32_t n_sig, const int32_t* h_idx_in,
                         const void* h_q_fresh, const void* h_k_fresh, const void* h_v_fresh,
                         void* h_kv_k, void* h_kv_v, int32_t copy_back_kv,
                         void* h_hidden, int32_t* h_idx_out,
                         void* arena, size_t arena_bytes, void* stream);
int daf_layer_host_end(const daf_params* p, void* arena, size_t arena_bytes, void* stream);

/* Validation of caller-given positions (no counterpart in the paper).  daf_select and daf_layer trust idx_in to be
 * strictly increasing positions in [0, L_d): only then is "causal in packed order" the same as "causal by position"
 * (out-of-range positions are skipped and reported by the gather; an unsorted list is not noticed there).  This call
 * checks k positions on the device and records the first offence in the status word of `workspace` (at least 256
 * bytes, e.g. the layer workspace): daf_poll_status then returns DAF_ERR_BOUNDS.  Nothing faults or traps. */
int daf_check_indices(const daf_params* p, int32_t k, const int32_t* idx, void* workspace, size_t workspace_bytes,
                      void* stream);

/* Reads the device status word kept in `workspace` (synchronises `stream`):
 * DAF_OK, DAF_ERR_TIMEOUT or DAF_ERR_BOUNDS; the word is cleared. */
int daf_poll_status(void* workspace, void* stream);

/* Self-test of the failure path (no counterpart in the paper): launches one small CTA that waits, with the
 * same bounded wait all kernels of this library use, on a barrier that nothing ever signals.  The wait gives
 * up after `limit_ms` milliseconds (1..1000), the CTA records DAF_ERR_TIMEOUT in the status word of
 * `workspace` (device memory, at least 256 bytes, e.g. a layer workspace) and returns normally: nothing
 * traps and the context stays usable.  daf_poll_status then returns DAF_ERR_TIMEOUT once.  Returns DAF_OK
 * when the launch was enqueued; DAF_ERR_WORKSPACE / DAF_ERR_INVALID_ARG for a missing workspace or a
 * limit outside the range. */
int daf_selftest_bounded_wait(void* workspace, size_t workspace_bytes, int32_t limit_ms, void* stream);

/* Text for a daf_status; the numeric cudaError_t behind the last DAF_ERR_CUDA of this thread. */
const char* daf_strerror(int status);
int daf_last_cuda_error(void);

/* Number of kernels this library has launched in this process (for accounting). */
int64_t daf_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DAF_H_ */
