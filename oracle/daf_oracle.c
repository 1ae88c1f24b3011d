/*
 * CPU oracle for the prefill-attention path of Decoupled Attention Fusion (DAF).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * library is checked against.  It shares no code, header, table or helper with
 * the CUDA path, and nothing on the product path may call it.
 *
 * What it follows (paper sections, restated):
 *   - Methods, item 1 (selection + important-token self-attention): a fraction r
 *     of the L_d document tokens is picked from an importance signal aggregated
 *     over several layers, gathered into one condensed sequence, and attention
 *     is computed among those tokens only.
 *   - Methods, item 2 (question-document attention): the L_q question rows
 *     attend over all L_d + L_q keys, the document part of which is the hybrid
 *     cache (offline rows, with the important rows already replaced by fresh ones).
 *   - Methods, item 3 (state fusion): both outputs are concatenated into the
 *     compact hidden-state rows (or scattered back by position).
 *   - Full recomputation (the comparison system's attention): causal attention
 *     over all L_d + L_q fresh rows.
 *
 * Arithmetic: inputs are fp32 arrays that hold bf16-representable values (the
 * caller widens, which is exact).  Every dot product, the softmax and the
 * weighted sum are carried in fp64; results are returned in fp64 so that the
 * caller decides on the comparison precision.  The softmax is the two-pass
 * textbook form (row maximum, then exponentials and their sum); there is no
 * tiling, no online rescaling, no reordering.
 *
 * Pins (see tests/test_oracle_*.py): the attention routine is checked against a
 * library attention (torch scaled_dot_product_attention, fp64, causal), against
 * closed forms (zero keys -> running mean of V, constant V, one visible key,
 * hand-worked rational example in tests/golden/), against a brute-force masked
 * N x N attention over the concatenated context, and the selection against a
 * library stable argsort and an O(L_d^2) rank count.
 * The fp8 decode is pinned against a library conversion of all 256 byte values and stated values of the
 * format (largest finite 448, smallest subnormal 2^-9), the expansion by "scale 1 == widening".
 * Parity unpinned: the *formula* of the per-layer deviation signal (the paper names
 * the signal but gives no formula; daf_oracle_deviation_scores states the reading
 * taken).  The selection rule applied to given scores is pinned, and so is the
 * arithmetic of the chosen deviation formula.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* Number of important tokens for a fraction r of L_d document tokens
 * (Methods, notation paragraph: r, the share of the document tokens that is recomputed).
 * Reading: k = ceil(r * L_d), clamped to [0, L_d].  The product is shrunk by a
 * relative 1e-6 before the ceiling so that an r that was rounded to single
 * precision (0.1f * 1000 = 100.0000015) still gives the intended count. */
int64_t daf_oracle_num_important(int64_t L_d, double r)
{
    if (L_d <= 0 || !(r > 0.0)) return 0;
    double x = ceil(r * (double)L_d * (1.0 - 1e-6));
    if (x < 0.0) x = 0.0;
    if (x > (double)L_d) x = (double)L_d;
    return (int64_t)x;
}

/* Aggregated importance signal (Methods, item 1: signals from several layers
 * are aggregated).  Reading: plain sum over the signal rows, added in ascending
 * row order, in fp32 (the precision in which the ranking decision is taken). */
void daf_oracle_aggregate(const float *S, int32_t n_sig, int32_t L_d, float *s_out)
{
    for (int32_t i = 0; i < L_d; ++i) {
        float acc = S[i];
        for (int32_t l = 1; l < n_sig; ++l) acc = acc + S[(int64_t)l * L_d + i];
        s_out[i] = acc;
    }
}

typedef struct { float s; int32_t i; } scored_t;

/* Total order used for selection: higher score first; equal scores (+0 == -0)
 * by lower index first; NaN ranks below every number. */
static int scored_before(const void *pa, const void *pb)
{
    const scored_t *a = (const scored_t *)pa, *b = (const scored_t *)pb;
    int an = isnan(a->s), bn = isnan(b->s);
    if (an != bn) return an ? 1 : -1;
    if (!an) {
        if (a->s > b->s) return -1;
        if (a->s < b->s) return 1;
    }
    return (a->i > b->i) - (a->i < b->i);
}

static int int32_ascending(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/* Important-token selection (Methods, item 1): the k highest aggregated scores,
 * reported as token positions in ascending order.  This is the definition
 * itself: sort every index by the total order, keep the first k. */
int32_t daf_oracle_select(const float *S, int32_t n_sig, int32_t L_d, int32_t k, int32_t *idx_out)
{
    if (k < 0 || k > L_d || n_sig < 1) return -1;
    float *s = (float *)malloc(sizeof(float) * (size_t)(L_d > 0 ? L_d : 1));
    scored_t *e = (scored_t *)malloc(sizeof(scored_t) * (size_t)(L_d > 0 ? L_d : 1));
    if (!s || !e) { free(s); free(e); return -2; }
    daf_oracle_aggregate(S, n_sig, L_d, s);
    for (int32_t i = 0; i < L_d; ++i) { e[i].s = s[i]; e[i].i = i; }
    qsort(e, (size_t)L_d, sizeof(scored_t), scored_before);
    for (int32_t j = 0; j < k; ++j) idx_out[j] = e[j].i;
    qsort(idx_out, (size_t)k, sizeof(int32_t), int32_ascending);
    free(s); free(e);
    return 0;
}

/* Condensed sequence (Methods, item 1: important tokens are gathered into a
 * condensed sequence): dst[j] = src[idx[j]], rows of row_elems values. */
void daf_oracle_gather_rows(const float *src, const int32_t *idx, int32_t k, int64_t row_elems, float *dst)
{
    for (int32_t j = 0; j < k; ++j)
        memcpy(dst + (int64_t)j * row_elems, src + (int64_t)idx[j] * row_elems, sizeof(float) * (size_t)row_elems);
}

/* Hybrid KV cache (Methods, item 2): document rows come from the offline cache,
 * except the important rows, which are replaced by their fresh values; the
 * question rows L_d .. L_d+L_q-1 are the fresh question rows.
 * overwrite == 0 leaves the document rows offline (ablation of that reading). */
void daf_oracle_hybrid_kv(const float *cached, const float *fresh, const int32_t *idx, int32_t k,
                          int32_t L_d, int32_t L_q, int64_t row_elems, int32_t overwrite, float *hybrid)
{
    memcpy(hybrid, cached, sizeof(float) * (size_t)((int64_t)L_d * row_elems));
    if (overwrite)
        for (int32_t j = 0; j < k; ++j)
            memcpy(hybrid + (int64_t)idx[j] * row_elems, fresh + (int64_t)idx[j] * row_elems,
                   sizeof(float) * (size_t)row_elems);
    memcpy(hybrid + (int64_t)L_d * row_elems, fresh + (int64_t)L_d * row_elems,
           sizeof(float) * (size_t)((int64_t)L_q * row_elems));
}

/* Softmax attention of selected query rows, grouped-query heads, causal with an
 * offset: query row p sees keys t <= p + offset (and t < n_kv); when `last_key` is
 * given, row p sees keys t <= last_key[p] instead.
 *   q   [n_q , Hq , D]   k, v [n_kv, Hkv, D]   token-major, fp32 values
 *   rows: n_rows query-row numbers to evaluate, or NULL for rows 0..n_rows-1
 *   out [n_rows, Hq, D] fp64;  lse [n_rows, Hq] fp64 (may be NULL)
 * Query head h reads KV head h / (Hq / Hkv). */
static void attention_rows(const float *q, const float *k, const float *v,
                           int32_t n_q, int32_t n_kv, int32_t Hq, int32_t Hkv, int32_t D,
                           double scale, int64_t offset, const int32_t *last_key,
                           const int32_t *rows, int32_t n_rows, double *out, double *lse)
{
    const int32_t G = Hq / Hkv;
    (void)n_q;
#pragma omp parallel
    {
        double *logit = (double *)malloc(sizeof(double) * (size_t)(n_kv > 0 ? n_kv : 1));
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int32_t a = 0; a < n_rows; ++a) {
            for (int32_t h = 0; h < Hq; ++h) {
                const int32_t p = rows ? rows[a] : a;
                const int32_t g = h / G;
                int64_t n_vis = last_key ? (int64_t)last_key[p] + 1 : (int64_t)p + offset + 1;
                if (n_vis > n_kv) n_vis = n_kv;
                double *o = out + ((int64_t)a * Hq + h) * D;
                for (int32_t d = 0; d < D; ++d) o[d] = 0.0;
                if (n_vis <= 0) { if (lse) lse[(int64_t)a * Hq + h] = -INFINITY; continue; }
                const float *qr = q + ((int64_t)p * Hq + h) * D;
                double m = -INFINITY;
                for (int64_t t = 0; t < n_vis; ++t) {
                    const float *kr = k + (t * Hkv + g) * D;
                    double acc = 0.0;
                    for (int32_t d = 0; d < D; ++d) acc += (double)qr[d] * (double)kr[d];
                    acc *= scale;
                    logit[t] = acc;
                    if (acc > m) m = acc;
                }
                double l = 0.0;
                for (int64_t t = 0; t < n_vis; ++t) {
                    double e = exp(logit[t] - m);
                    logit[t] = e;
                    l += e;
                }
                for (int64_t t = 0; t < n_vis; ++t) {
                    const float *vr = v + (t * Hkv + g) * D;
                    const double w = logit[t];
                    for (int32_t d = 0; d < D; ++d) o[d] += w * (double)vr[d];
                }
                for (int32_t d = 0; d < D; ++d) o[d] /= l;
                if (lse) lse[(int64_t)a * Hq + h] = m + log(l);
            }
        }
        free(logit);
    }
}

/* Important-token self-attention (Methods, item 1; cost term r^2 L_d^2 of the
 * complexity analysis): attention among the k packed rows only.  Reading:
 * causal in packed order, which equals causal by original position because the
 * packed rows are in ascending position order. */
void daf_oracle_important_attn(const float *q_pack, const float *k_pack, const float *v_pack,
                               int32_t k, int32_t Hq, int32_t Hkv, int32_t D, double scale,
                               const int32_t *rows, int32_t n_rows, double *out, double *lse)
{
    attention_rows(q_pack, k_pack, v_pack, k, k, Hq, Hkv, D, scale, 0, NULL, rows, n_rows, out, lse);
}

/* Question-document attention (Methods, item 2): an L_q x (L_d + L_q) attention;
 * question row i sits at position L_d + i and sees every hybrid-cache key up to
 * and including itself. */
void daf_oracle_qd_attn(const float *q_question, const float *kv_k, const float *kv_v,
                        int32_t L_d, int32_t L_q, int32_t Hq, int32_t Hkv, int32_t D, double scale,
                        const int32_t *rows, int32_t n_rows, double *out, double *lse)
{
    attention_rows(q_question, kv_k, kv_v, L_q, L_d + L_q, Hq, Hkv, D, scale, L_d, NULL, rows, n_rows, out, lse);
}

/* Full recomputation (the comparison path of the experiments): causal attention
 * over all n fresh rows. */
void daf_oracle_full_causal_attn(const float *q, const float *k, const float *v,
                                 int32_t n, int32_t Hq, int32_t Hkv, int32_t D, double scale,
                                 const int32_t *rows, int32_t n_rows, double *out, double *lse)
{
    attention_rows(q, k, v, n, n, Hq, Hkv, D, scale, 0, NULL, rows, n_rows, out, lse);
}

/* Selective recomputation over the full context (Complexity Analysis: the scheme DAF is
 * compared with lets the important rows and the question rows attend the whole context, at a
 * cost of about r L_d^2 + L_d L_q, against r^2 L_d^2 + L_q (L_d + L_q) for DAF).  The compact
 * rows (important rows in position order, then the question rows) each attend every key of
 * the hybrid cache up to their own position row_pos[j].  Built only to measure that cost
 * ratio on the same kernels; it is not part of the DAF path. */
void daf_oracle_blend_attn(const float *q_rows, const float *kv_k, const float *kv_v, const int32_t *row_pos,
                           int32_t n_q, int32_t n_kv, int32_t Hq, int32_t Hkv, int32_t D, double scale,
                           const int32_t *rows, int32_t n_rows, double *out, double *lse)
{
    attention_rows(q_rows, kv_k, kv_v, n_q, n_kv, Hq, Hkv, D, scale, 0, row_pos, rows, n_rows, out, lse);
}

/* Per-layer importance signal (Methods, item 1: important tokens are found from the
 * deviation between the freshly computed and the offline KV states of a layer).  The
 * paper names the signal but prints no formula; the reading taken here is the squared
 * Euclidean deviation of a token's K and V rows, summed over heads and channels:
 *   s[i] = sum_{h,d} (Kf[i,h,d] - Kc[i,h,d])^2 + (Vf[i,h,d] - Vc[i,h,d])^2 .
 * Parity unpinned as far as the choice of formula goes; the arithmetic of this
 * formula is pinned (zero for equal tensors, c^2 for one element off by c, a
 * hand-worked case, a library sum of squares). */
void daf_oracle_deviation_scores(const float *k_fresh, const float *v_fresh, const float *k_cached,
                                 const float *v_cached, int32_t L_d, int64_t row_elems, double *s_out)
{
#pragma omp parallel for schedule(static)
    for (int32_t i = 0; i < L_d; ++i) {
        double acc = 0.0;
        for (int64_t e = 0; e < row_elems; ++e) {
            const double dk = (double)k_fresh[(int64_t)i * row_elems + e] - (double)k_cached[(int64_t)i * row_elems + e];
            const double dv = (double)v_fresh[(int64_t)i * row_elems + e] - (double)v_cached[(int64_t)i * row_elems + e];
            acc += dk * dk + dv * dv;
        }
        s_out[i] = acc;
    }
}

/* ------------------------------------------------- offline cache stored in fp8
 * (Preliminary Results, Limitations: the storage of the offline KV caches is the
 * industrial bottleneck.)  Reading taken for the stored-in-fp8 variant: an offline
 * K or V element is one byte in the 8-bit floating-point format with 1 sign bit,
 * 4 exponent bits (bias 7) and 3 mantissa bits, no infinities, and the single
 * NaN pattern S.1111.111 ("e4m3"); every KV head has one fp32 scale.  The value
 * the attention sees is   bf16( scale * decode(byte) )   with the product taken in
 * fp32 and both roundings to nearest-even: the cache is expanded to the bf16
 * working precision of the rest of the path, after which nothing differs from the
 * bf16 path.  With scale = 1 the expansion is exact (every e4m3 value is a bf16
 * value).
 */
float daf_oracle_e4m3_decode(uint8_t byte)
{
    const int sign = byte >> 7, e = (byte >> 3) & 0xF, m = byte & 0x7;
    float v;
    if (e == 0xF && m == 0x7) return NAN;
    if (e == 0) v = ldexpf((float)m, -9);                 /* subnormal: m/8 * 2^-6 */
    else v = ldexpf(1.0f + (float)m / 8.0f, e - 7);
    return sign ? -v : v;
}

static float round_to_bf16(float x)
{
    uint32_t u;
    memcpy(&u, &x, 4);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return x;        /* NaN stays NaN */
    u += 0x7FFFu + ((u >> 16) & 1u);                      /* round to nearest, ties to even */
    u &= 0xFFFF0000u;
    memcpy(&x, &u, 4);
    return x;
}

/* bytes: [tokens, heads, D] e4m3; scale: [heads] or NULL (all 1); out: fp32 [tokens, heads, D]
 * holding bf16-representable values. */
void daf_oracle_dequant_fp8(const uint8_t *bytes, const float *scale, int64_t tokens, int32_t heads, int32_t D,
                            float *out)
{
    for (int64_t t = 0; t < tokens; ++t)
        for (int32_t h = 0; h < heads; ++h) {
            const float s = scale ? scale[h] : 1.0f;
            for (int32_t d = 0; d < D; ++d) {
                const int64_t i = (t * heads + h) * D + d;
                const float prod = s * daf_oracle_e4m3_decode(bytes[i]);    /* fp32 product, rounded once */
                out[i] = round_to_bf16(prod);
            }
        }
}

/* State fusion (Methods, item 3).  mode 0: compact concatenation, important rows
 * first then question rows (position order).  mode 1: scatter to the original
 * positions of an (L_d+L_q)-row buffer whose other rows are left untouched.
 * row_pos_out (optional, k+L_q entries) receives the original position of each
 * compact row. */
void daf_oracle_fuse(const double *o_imp, const double *o_q, const int32_t *idx, int32_t k,
                     int32_t L_d, int32_t L_q, int64_t row_elems, int32_t mode,
                     double *hidden, int32_t *row_pos_out)
{
    for (int32_t j = 0; j < k + L_q; ++j) {
        const int32_t pos = j < k ? idx[j] : L_d + (j - k);
        const double *src = j < k ? o_imp + (int64_t)j * row_elems : o_q + (int64_t)(j - k) * row_elems;
        const int64_t dst_row = mode == 0 ? j : pos;
        memcpy(hidden + dst_row * row_elems, src, sizeof(double) * (size_t)row_elems);
        if (row_pos_out) row_pos_out[j] = pos;
    }
}

int32_t daf_oracle_num_threads(void)
{
#ifdef _OPENMP
    return (int32_t)omp_get_max_threads();
#else
    return 1;
#endif
}
