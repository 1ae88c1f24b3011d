// C ABI of the DAF library (see include/daf.h): argument validation, workspace
// carving and the order of launches.  No arithmetic of the method lives here.
#include <atomic>
#include <math.h>
#include <string.h>

#include "daf_common.cuh"

namespace daf {

static thread_local int g_last_cuda_error = 0;
static std::atomic<long long> g_launches{0};

void set_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
int check_launch() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
    return DAF_OK;
}

static int num_important(int L_d, double r) {
    if (L_d <= 0 || !(r > 0.0)) return 0;
    double x = ceil(r * (double)L_d * (1.0 - 1e-6));
    if (x < 0.0) x = 0.0;
    if (x > (double)L_d) x = (double)L_d;
    return (int)x;
}

constexpr int kMaxTokens = 1 << 22;   // 4M rows: keeps every 32-bit index product in range
constexpr int kMaxHeads = 256;

int resolve_params(const daf_params* p, ResolvedParams* out) {
    if (p == nullptr) return DAF_ERR_INVALID_ARG;
    if (p->L_d < 0 || p->L_q < 0) return DAF_ERR_INVALID_ARG;
    if (!(p->r >= 0.0) || p->r > 1.0) return DAF_ERR_INVALID_ARG;
    if (p->n_q_heads <= 0 || p->n_kv_heads <= 0) return DAF_ERR_INVALID_ARG;
    if (p->fuse_mode != 0 && p->fuse_mode != 1) return DAF_ERR_INVALID_ARG;
    if (p->head_dim != 128) return DAF_ERR_UNSUPPORTED;
    if (p->n_q_heads % p->n_kv_heads != 0) return DAF_ERR_UNSUPPORTED;
    if (p->n_q_heads > kMaxHeads) return DAF_ERR_UNSUPPORTED;
    if ((long long)p->L_d + p->L_q > kMaxTokens) return DAF_ERR_UNSUPPORTED;
    out->L_d = p->L_d; out->L_q = p->L_q; out->N = p->L_d + p->L_q;
    out->Hq = p->n_q_heads; out->Hkv = p->n_kv_heads; out->G = out->Hq / out->Hkv;
    out->k = num_important(p->L_d, p->r);
    out->scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
    out->fuse_mode = p->fuse_mode;
    out->overwrite = p->overwrite_doc_kv != 0;
    return DAF_OK;
}

struct Workspace {
    DeviceStatus* status;
    float* signal_sums;       // [L_d] aggregated importance signal (daf_select_from_kv)
    void* select_scratch;
    void* attn_scratch;
    size_t attn_bytes;
};

static size_t qd_partial_bytes(const ResolvedParams& rp) {
    if (rp.L_q == 0) return 0;
    AttnPlan pl = plan_attention(rp.L_q, rp.N, rp.Hq, rp.G, rp.L_d, true, true);
    return attn_partial_bytes(rp.L_q, rp.Hq, pl.n_splits);
}

// The attention scratch serves the stand-alone question stage and the joint launch of steps 2 and 3.
static size_t attn_scratch_bytes(const ResolvedParams& rp) {
    size_t need = qd_partial_bytes(rp);
    if (rp.k > 0 && rp.L_q > 0) {
        const size_t joint = joint_partial_bytes(plan_joint(rp.k, rp.L_q, rp.L_d, rp.Hq, rp.G));
        if (joint > need) need = joint;
    }
    return need;
}

static size_t signal_sum_bytes(const ResolvedParams& rp) { return ((size_t)rp.L_d * sizeof(float) + 255) / 256 * 256; }

static size_t workspace_bytes(const ResolvedParams& rp) {
    return kStatusBytes + signal_sum_bytes(rp) + select_scratch_bytes(rp.L_d) + attn_scratch_bytes(rp);
}

static int carve_workspace(const ResolvedParams& rp, void* workspace, size_t bytes, Workspace* ws) {
    if (workspace == nullptr || bytes < workspace_bytes(rp)) return DAF_ERR_WORKSPACE;
    if (!aligned16(workspace)) return DAF_ERR_ALIGNMENT;
    char* base = reinterpret_cast<char*>(workspace);
    ws->status = reinterpret_cast<DeviceStatus*>(base);
    ws->signal_sums = reinterpret_cast<float*>(base + kStatusBytes);
    ws->select_scratch = base + kStatusBytes + signal_sum_bytes(rp);
    ws->attn_scratch = base + kStatusBytes + signal_sum_bytes(rp) + select_scratch_bytes(rp.L_d);
    ws->attn_bytes = bytes - kStatusBytes - signal_sum_bytes(rp) - select_scratch_bytes(rp.L_d);
    return DAF_OK;
}

static int do_select(const ResolvedParams& rp, const float* scores, int32_t n_sig, const int32_t* idx_in,
                     const void* q_fresh, const void* k_fresh, const void* v_fresh, void* kv_k, void* kv_v,
                     int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack, const Workspace& ws, cudaStream_t st,
                     bool scores_from_previous_kernel = false, bool beside_previous_kernel = false, bool rows_far = false) {
    if (scores != nullptr && n_sig < 1) return DAF_ERR_INVALID_ARG;
    if (rp.k > 0) {
        if (scores == nullptr && idx_in == nullptr) return DAF_ERR_INVALID_ARG;
        if (scores != nullptr && idx_out == nullptr) return DAF_ERR_INVALID_ARG;
        if (!q_fresh || !k_fresh || !v_fresh) return DAF_ERR_INVALID_ARG;   // q_pack is optional
        if ((k_pack == nullptr) != (v_pack == nullptr)) return DAF_ERR_INVALID_ARG;   // k_pack / v_pack: both or neither
        if (rp.overwrite && (!kv_k || !kv_v)) return DAF_ERR_INVALID_ARG;
    }
    if (rp.L_q > 0 && (!k_fresh || !v_fresh || !kv_k || !kv_v)) return DAF_ERR_INVALID_ARG;
    if (kv_k != nullptr && (kv_k == k_fresh || kv_v == v_fresh)) return DAF_ERR_INVALID_ARG;
    const void* ptrs[] = {scores, idx_in, q_fresh, k_fresh, v_fresh, kv_k, kv_v, idx_out, q_pack, k_pack, v_pack};
    for (const void* ptr : ptrs)
        if (ptr != nullptr && !aligned16(ptr)) return DAF_ERR_ALIGNMENT;
    return launch_select(rp, scores, n_sig, idx_in, q_fresh, k_fresh, v_fresh, kv_k, kv_v, idx_out, q_pack, k_pack,
                         v_pack, ws.status, ws.select_scratch, st, scores_from_previous_kernel, beside_previous_kernel,
                         /*select_only=*/false, rows_far);
}

static int check_out(const void* out, int64_t stride_bytes, int Hq) {
    if (out == nullptr) return DAF_ERR_INVALID_ARG;
    if (!aligned16(out) || stride_bytes % 16 != 0) return DAF_ERR_ALIGNMENT;
    if (stride_bytes < (int64_t)Hq * 256) return DAF_ERR_INVALID_ARG;
    return DAF_OK;
}

}  // namespace daf

using namespace daf;

#define DAF_CUDA_TRY(expr)                                                \
    do {                                                                  \
        cudaError_t e_ = (expr);                                          \
        if (e_ != cudaSuccess) { set_cuda_error(e_); return DAF_ERR_CUDA; } \
    } while (0)

extern "C" {

int32_t daf_num_important(int32_t L_d, double r) { return num_important(L_d, r); }

size_t daf_workspace_bytes(const daf_params* p) {
    ResolvedParams rp;
    if (resolve_params(p, &rp) != DAF_OK) return 0;
    return workspace_bytes(rp);
}

int daf_select(const daf_params* p, const float* scores, int32_t n_sig, const int32_t* idx_in,
               const void* q_fresh, const void* k_fresh, const void* v_fresh, void* kv_k, void* kv_v,
               int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack,
               void* workspace, size_t workspace_bytes_, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    Workspace ws;
    if (int rc = carve_workspace(rp, workspace, workspace_bytes_, &ws)) return rc;
    return do_select(rp, scores, n_sig, idx_in, q_fresh, k_fresh, v_fresh, kv_k, kv_v, idx_out, q_pack, k_pack, v_pack,
                     ws, (cudaStream_t)stream);
}

int daf_select_from_kv(const daf_params* p, int32_t n_sig, const void* const* sig_k_fresh, const void* const* sig_v_fresh,
                       const void* const* sig_k_cached, const void* const* sig_v_cached,
                       const void* q_fresh, const void* k_fresh, const void* v_fresh, void* kv_k, void* kv_v,
                       int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack, float* signal_sum_out,
                       void* workspace, size_t workspace_bytes_, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    Workspace ws;
    if (int rc = carve_workspace(rp, workspace, workspace_bytes_, &ws)) return rc;
    if (n_sig < 1 || n_sig > kMaxSignalLayersHost) return DAF_ERR_INVALID_ARG;
    if (!sig_k_fresh || !sig_v_fresh || !sig_k_cached || !sig_v_cached) return DAF_ERR_INVALID_ARG;
    for (int l = 0; l < n_sig; ++l) {
        const void* ptrs[] = {sig_k_fresh[l], sig_v_fresh[l], sig_k_cached[l], sig_v_cached[l]};
        for (const void* ptr : ptrs) {
            if (ptr == nullptr) return DAF_ERR_INVALID_ARG;
            if (!aligned16(ptr)) return DAF_ERR_ALIGNMENT;
        }
    }
    if (signal_sum_out != nullptr && (reinterpret_cast<uintptr_t>(signal_sum_out) & 15u) != 0) return DAF_ERR_ALIGNMENT;
    if (rp.k > 0 && idx_out == nullptr) return DAF_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    float* sums = signal_sum_out != nullptr ? signal_sum_out : ws.signal_sums;
    if (rp.L_d > 0)
        if (int rc = launch_deviation_sum(rp, n_sig, sig_k_fresh, sig_v_fresh, sig_k_cached, sig_v_cached, sums, st)) return rc;
    // the sums are one signal row: from here on this is daf_select, launched right behind the signal kernel
    return do_select(rp, rp.L_d > 0 ? sums : nullptr, 1, nullptr, q_fresh, k_fresh, v_fresh, kv_k, kv_v, idx_out, q_pack, k_pack,
                     v_pack, ws, st, /*scores_from_previous_kernel=*/true);
}

int daf_important_attn(const daf_params* p, int32_t k, const void* q_pack, const void* k_pack, const void* v_pack,
                       void* out, int64_t out_row_stride_bytes, const int32_t* dst_rows, float* lse,
                       void* workspace, size_t workspace_bytes_, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    if (k < 0 || k > rp.L_d) return DAF_ERR_INVALID_ARG;
    Workspace ws;
    if (int rc = carve_workspace(rp, workspace, workspace_bytes_, &ws)) return rc;
    if (k == 0) return DAF_OK;
    if (!q_pack || !k_pack || !v_pack) return DAF_ERR_INVALID_ARG;
    if (!aligned16(q_pack) || !aligned16(k_pack) || !aligned16(v_pack)) return DAF_ERR_ALIGNMENT;
    if (int rc = check_out(out, out_row_stride_bytes, rp.Hq)) return rc;
    return launch_attention(q_pack, k_pack, v_pack, k, k, rp.Hq, rp.Hkv, 0, rp.scale, false, false, out,
                            out_row_stride_bytes, dst_rows, lse, ws.status, ws.attn_scratch, ws.attn_bytes,
                            (cudaStream_t)stream);
}

int daf_qd_attn(const daf_params* p, const void* q_question, const void* kv_k, const void* kv_v,
                void* out, int64_t out_row_stride_bytes, const int32_t* dst_rows, float* lse,
                void* workspace, size_t workspace_bytes_, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    Workspace ws;
    if (int rc = carve_workspace(rp, workspace, workspace_bytes_, &ws)) return rc;
    if (rp.L_q == 0) return DAF_OK;
    if (!q_question || !kv_k || !kv_v) return DAF_ERR_INVALID_ARG;
    if (!aligned16(q_question) || !aligned16(kv_k) || !aligned16(kv_v)) return DAF_ERR_ALIGNMENT;
    if (int rc = check_out(out, out_row_stride_bytes, rp.Hq)) return rc;
    return launch_attention(q_question, kv_k, kv_v, rp.L_q, rp.N, rp.Hq, rp.Hkv, rp.L_d, rp.scale, true, true, out,
                            out_row_stride_bytes, dst_rows, lse, ws.status, ws.attn_scratch, ws.attn_bytes,
                            (cudaStream_t)stream);
}

int daf_imp_qd_attn(const daf_params* p, const void* q_pack, const void* q_fresh, const void* k_pack, const void* v_pack,
                    const void* q_question, const void* kv_k, const void* kv_v, const int32_t* idx,
                    void* hidden, void* workspace, size_t workspace_bytes_, void* stream) {
    return daf_imp_qd_attn_launches(p, q_pack, q_fresh, k_pack, v_pack, q_question, kv_k, kv_v, idx, hidden, workspace,
                                    workspace_bytes_, stream, 3);
}

int daf_imp_qd_attn_launches(const daf_params* p, const void* q_pack, const void* q_fresh, const void* k_pack, const void* v_pack,
                             const void* q_question, const void* kv_k, const void* kv_v, const int32_t* idx,
                             void* hidden, void* workspace, size_t workspace_bytes_, void* stream, int32_t launches) {
    if (launches < 1 || launches > 3) return DAF_ERR_INVALID_ARG;
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    Workspace ws;
    if (int rc = carve_workspace(rp, workspace, workspace_bytes_, &ws)) return rc;
    if (rp.k <= 0 || rp.L_q <= 0) return DAF_ERR_INVALID_ARG;
    if (!k_pack || !v_pack || !q_question || !kv_k || !kv_v) return DAF_ERR_INVALID_ARG;
    if (q_pack == nullptr && (q_fresh == nullptr || idx == nullptr)) return DAF_ERR_INVALID_ARG;
    if (rp.fuse_mode == 1 && idx == nullptr) return DAF_ERR_INVALID_ARG;
    const void* ptrs[] = {q_pack, q_fresh, k_pack, v_pack, q_question, kv_k, kv_v, idx};
    for (const void* ptr : ptrs)
        if (ptr != nullptr && !aligned16(ptr)) return DAF_ERR_ALIGNMENT;
    const int64_t row_bytes = (int64_t)rp.Hq * 256;
    if (int rc = check_out(hidden, row_bytes, rp.Hq)) return rc;
    char* h = reinterpret_cast<char*>(hidden);
    const int64_t first_row = rp.fuse_mode == 1 ? rp.L_d : rp.k;
    return launch_attention_joint(q_pack, q_fresh, idx, k_pack, v_pack, nullptr, nullptr, rp.k, h, rp.fuse_mode == 1 ? idx : nullptr, q_question, kv_k, kv_v,
                                  rp.L_q, rp.L_d, h + first_row * row_bytes, row_bytes, rp.Hq, rp.Hkv, rp.scale, ws.status,
                                  ws.attn_scratch, ws.attn_bytes, (cudaStream_t)stream, /*after_kernel=*/false, launches);
}

int daf_blend_attn(const daf_params* p, int32_t n_rows, const void* q_rows, const void* kv_k, const void* kv_v,
                   const int32_t* row_pos, void* out, int64_t out_row_stride_bytes, float* lse,
                   void* workspace, size_t workspace_bytes_, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    if (n_rows < 0 || n_rows > rp.N) return DAF_ERR_INVALID_ARG;
    Workspace ws;
    if (int rc = carve_workspace(rp, workspace, workspace_bytes_, &ws)) return rc;
    if (n_rows == 0) return DAF_OK;
    if (!q_rows || !kv_k || !kv_v || !row_pos) return DAF_ERR_INVALID_ARG;
    if (!aligned16(q_rows) || !aligned16(kv_k) || !aligned16(kv_v) || (reinterpret_cast<uintptr_t>(row_pos) & 3u)) return DAF_ERR_ALIGNMENT;
    if (int rc = check_out(out, out_row_stride_bytes, rp.Hq)) return rc;
    // causal_off = N - n_rows only sizes the launch (last row sees at most N keys); the limits come from row_pos
    return launch_attention(q_rows, kv_k, kv_v, n_rows, rp.N, rp.Hq, rp.Hkv, rp.N - n_rows, rp.scale, false, false, out,
                            out_row_stride_bytes, nullptr, lse, ws.status, ws.attn_scratch, ws.attn_bytes,
                            (cudaStream_t)stream, false, row_pos);
}

int daf_deviation_scores(const daf_params* p, const void* k_fresh, const void* v_fresh, const void* k_cached,
                         const void* v_cached, float* scores_row, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    if (rp.L_d == 0) return DAF_OK;
    if (!k_fresh || !v_fresh || !k_cached || !v_cached || !scores_row) return DAF_ERR_INVALID_ARG;
    if (!aligned16(k_fresh) || !aligned16(v_fresh) || !aligned16(k_cached) || !aligned16(v_cached) ||
        (reinterpret_cast<uintptr_t>(scores_row) & 3u) != 0) return DAF_ERR_ALIGNMENT;
    return launch_deviation_scores(rp, k_fresh, v_fresh, k_cached, v_cached, scores_row, (cudaStream_t)stream);
}

int daf_fuse(const daf_params* p, int32_t k, const int32_t* idx, const void* o_imp, const void* o_q,
             void* hidden, int32_t* row_pos_out, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    if (k < 0 || k > rp.L_d) return DAF_ERR_INVALID_ARG;
    rp.k = k;
    if (hidden == nullptr && row_pos_out == nullptr) return DAF_ERR_INVALID_ARG;
    if (k > 0 && (idx == nullptr || (hidden != nullptr && o_imp == nullptr))) return DAF_ERR_INVALID_ARG;
    if (rp.L_q > 0 && hidden != nullptr && o_q == nullptr) return DAF_ERR_INVALID_ARG;
    if ((o_imp && !aligned16(o_imp)) || (o_q && !aligned16(o_q)) || (hidden && !aligned16(hidden))) return DAF_ERR_ALIGNMENT;
    return launch_fuse(rp, idx, o_imp, o_q, hidden, row_pos_out, (cudaStream_t)stream);
}

int daf_full_causal_attn(const daf_params* p, int32_t n_tokens, const void* q, const void* k, const void* v,
                         void* out, float* lse, void* workspace, size_t workspace_bytes_, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    if (n_tokens < 0 || n_tokens > kMaxTokens) return DAF_ERR_INVALID_ARG;
    Workspace ws;
    if (int rc = carve_workspace(rp, workspace, workspace_bytes_, &ws)) return rc;
    if (n_tokens == 0) return DAF_OK;
    if (!q || !k || !v) return DAF_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v)) return DAF_ERR_ALIGNMENT;
    if (int rc = check_out(out, (int64_t)rp.Hq * 256, rp.Hq)) return rc;
    return launch_attention(q, k, v, n_tokens, n_tokens, rp.Hq, rp.Hkv, 0, rp.scale, false, false, out,
                            (long long)rp.Hq * 256, nullptr, lse, ws.status, ws.attn_scratch, ws.attn_bytes,
                            (cudaStream_t)stream);
}

}  // extern "C"

namespace {
// Offline cache of one layer kept in fp8 (daf_layer_fp8): expanded into kv_k / kv_v ahead of everything else.
struct Fp8Cache { const void* k8; const void* v8; const float* k_scale; const float* v_scale; };
// Where the gather / cache-update kernel reads the fresh rows when that is not the tensors the attention reads the
// question rows from: device-accessible pointers to [N, heads, 128] tensors (mapped pinned host memory).
struct RowSource { const void* q; const void* k; const void* v; };

int layer_impl(const daf_params* p, const Fp8Cache* fp8, const float* scores, int32_t n_sig, const int32_t* idx_in,
               const void* q_fresh, const void* k_fresh, const void* v_fresh, void* kv_k, void* kv_v,
               int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack,
               void* hidden, int32_t* row_pos_out,
               void* workspace, size_t workspace_bytes_, void* stream, const RowSource* rows = nullptr) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    Workspace ws;
    if (int rc = carve_workspace(rp, workspace, workspace_bytes_, &ws)) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (rp.k + rp.L_q == 0) return DAF_OK;
    if (rows != nullptr && (q_pack == nullptr || k_pack == nullptr)) return DAF_ERR_INVALID_ARG;   // only the gather kernel reads them
    if (fp8 != nullptr) {
        if (rp.L_d > 0 && (!fp8->k8 || !fp8->v8 || !kv_k || !kv_v)) return DAF_ERR_INVALID_ARG;
        if (!aligned16(fp8->k8) || !aligned16(fp8->v8) || !aligned16(kv_k) || !aligned16(kv_v)) return DAF_ERR_ALIGNMENT;
    }
    if (rp.k > 0 && idx_out == nullptr) return DAF_ERR_INVALID_ARG;
    // only the joint launch reads the important rows in place
    if (rp.k > 0 && rp.L_q == 0 && (q_pack == nullptr || k_pack == nullptr || v_pack == nullptr)) return DAF_ERR_INVALID_ARG;
    // the question rows are read from q_fresh even when nothing is selected (r = 0)
    if (rp.L_q > 0 && (q_fresh == nullptr || kv_k == nullptr || kv_v == nullptr)) return DAF_ERR_INVALID_ARG;
    if (rp.k > 0 && (q_fresh == nullptr || (k_pack == nullptr) != (v_pack == nullptr))) return DAF_ERR_INVALID_ARG;
    if (q_fresh != nullptr && !aligned16(q_fresh)) return DAF_ERR_ALIGNMENT;
    const int64_t row_bytes = (int64_t)rp.Hq * 256;
    if (int rc = check_out(hidden, row_bytes, rp.Hq)) return rc;
    // An fp8 offline cache is expanded into the hybrid-cache buffer first.  The selection does not depend on it,
    // so the selection kernel is launched beside it; the gather kernel (which overwrites the important rows of
    // the expanded cache) runs behind both.
    if (fp8 != nullptr)
        if (int rc = launch_expand_fp8(rp, fp8->k8, fp8->v8, fp8->k_scale, fp8->v_scale, kv_k, kv_v, st)) return rc;
    if (int rc = do_select(rp, scores, n_sig, idx_in, rows ? rows->q : q_fresh, rows ? rows->k : k_fresh,
                           rows ? rows->v : v_fresh, kv_k, kv_v, idx_out, q_pack, k_pack,
                           v_pack, ws, st, false, /*beside_previous_kernel=*/fp8 != nullptr && rp.L_d > 0,
                           /*rows_far=*/rows != nullptr)) return rc;
    char* h = reinterpret_cast<char*>(hidden);
    // State fusion is done by the attention epilogues: each stage writes its final rows.  When both
    // stages have rows they run as one list of work items in one launch, right behind the gather
    // kernel of this call (the launch may overlap that kernel's tail).
    const int64_t first_row = rp.fuse_mode == 1 ? rp.L_d : rp.k;
    const char* qq = reinterpret_cast<const char*>(q_fresh) + (int64_t)rp.L_d * row_bytes;
    const int32_t* dst = rp.fuse_mode == 1 ? idx_out : nullptr;
    if (rp.k > 0 && rp.L_q > 0) {
        if (int rc = launch_attention_joint(q_pack, q_fresh, idx_out, k_pack, v_pack, k_fresh, v_fresh, rp.k, h, dst, qq, kv_k, kv_v, rp.L_q, rp.L_d,
                                            h + first_row * row_bytes, row_bytes, rp.Hq, rp.Hkv, rp.scale, ws.status,
                                            ws.attn_scratch, ws.attn_bytes, st, /*after_kernel=*/true)) return rc;
    } else if (rp.L_q > 0) {
        if (int rc = launch_attention(qq, kv_k, kv_v, rp.L_q, rp.N, rp.Hq, rp.Hkv, rp.L_d, rp.scale, true, true,
                                      h + first_row * row_bytes, row_bytes, nullptr, nullptr, ws.status, ws.attn_scratch,
                                      ws.attn_bytes, st, /*after_kernel=*/true)) return rc;
    } else {
        if (int rc = launch_attention(q_pack, k_pack, v_pack, rp.k, rp.k, rp.Hq, rp.Hkv, 0, rp.scale, false, false, h,
                                      row_bytes, dst, nullptr, ws.status, ws.attn_scratch, ws.attn_bytes, st,
                                      /*after_kernel=*/true)) return rc;
    }
    if (row_pos_out != nullptr) {
        if (int rc = launch_fuse(rp, idx_out, nullptr, nullptr, nullptr, row_pos_out, st)) return rc;
    }
    return DAF_OK;
}
}  // namespace

extern "C" {

int daf_layer(const daf_params* p, const float* scores, int32_t n_sig, const int32_t* idx_in,
              const void* q_fresh, const void* k_fresh, const void* v_fresh, void* kv_k, void* kv_v,
              int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack,
              void* hidden, int32_t* row_pos_out,
              void* workspace, size_t workspace_bytes_, void* stream) {
    return layer_impl(p, nullptr, scores, n_sig, idx_in, q_fresh, k_fresh, v_fresh, kv_k, kv_v, idx_out, q_pack, k_pack, v_pack,
                      hidden, row_pos_out, workspace, workspace_bytes_, stream);
}

int daf_layer_fp8(const daf_params* p, const float* scores, int32_t n_sig, const int32_t* idx_in,
                  const void* q_fresh, const void* k_fresh, const void* v_fresh,
                  const void* k_cached_fp8, const void* v_cached_fp8, const float* k_scale, const float* v_scale,
                  void* kv_k, void* kv_v, int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack,
                  void* hidden, int32_t* row_pos_out, void* workspace, size_t workspace_bytes_, void* stream) {
    const Fp8Cache fp8{k_cached_fp8, v_cached_fp8, k_scale, v_scale};
    return layer_impl(p, &fp8, scores, n_sig, idx_in, q_fresh, k_fresh, v_fresh, kv_k, kv_v, idx_out, q_pack, k_pack, v_pack,
                      hidden, row_pos_out, workspace, workspace_bytes_, stream);
}

int daf_select_topk(const daf_params* p, const float* scores, int32_t n_sig, int32_t* idx_out,
                    void* workspace, size_t workspace_bytes_, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    Workspace ws;
    if (int rc = carve_workspace(rp, workspace, workspace_bytes_, &ws)) return rc;
    if (rp.k == 0) return DAF_OK;
    if (scores == nullptr || idx_out == nullptr || n_sig < 1) return DAF_ERR_INVALID_ARG;
    if (!aligned16(scores) || !aligned16(idx_out)) return DAF_ERR_ALIGNMENT;
    // selection alone: no rows to gather, no question rows to append
    ResolvedParams sel = rp;
    sel.L_q = 0;
    return launch_select(sel, scores, n_sig, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, idx_out, nullptr, nullptr,
                         nullptr, ws.status, ws.select_scratch, (cudaStream_t)stream, false, false, /*select_only=*/true);
}

int daf_check_indices(const daf_params* p, int32_t k, const int32_t* idx, void* workspace, size_t workspace_bytes_,
                      void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    if (k < 0 || k > rp.L_d) return DAF_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes_ < kStatusBytes) return DAF_ERR_WORKSPACE;
    if (k == 0) return DAF_OK;
    if (idx == nullptr) return DAF_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(idx) & 3u) != 0 || !aligned16(workspace)) return DAF_ERR_ALIGNMENT;
    return launch_check_indices(idx, k, rp.L_d, reinterpret_cast<DeviceStatus*>(workspace), (cudaStream_t)stream);
}

int daf_expand_fp8_cache(const daf_params* p, const void* k_cached_fp8, const void* v_cached_fp8, const float* k_scale,
                         const float* v_scale, void* kv_k, void* kv_v, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    if (rp.L_d == 0) return DAF_OK;
    if (!k_cached_fp8 || !v_cached_fp8 || !kv_k || !kv_v) return DAF_ERR_INVALID_ARG;
    if (!aligned16(k_cached_fp8) || !aligned16(v_cached_fp8) || !aligned16(kv_k) || !aligned16(kv_v)) return DAF_ERR_ALIGNMENT;
    return launch_expand_fp8(rp, k_cached_fp8, v_cached_fp8, k_scale, v_scale, kv_k, kv_v, (cudaStream_t)stream);
}

// ---- host-buffer form
namespace {
struct Arena {
    char* ws; size_t ws_bytes;
    float* scores; int32_t* idx_in; int32_t* idx_out;
    char *q_fresh, *k_fresh, *v_fresh, *kv_k, *kv_v, *q_pack, *k_pack, *v_pack, *hidden;
    size_t total;
};
size_t up256(size_t x) { return (x + 255) / 256 * 256; }
void carve_arena(const ResolvedParams& rp, int n_sig, char* base, Arena* a) {
    size_t off = 0;
    auto take = [&](size_t bytes) { char* ptr = base ? base + off : nullptr; off += up256(bytes); return ptr; };
    const size_t qrow = (size_t)rp.Hq * 256, kvrow = (size_t)rp.Hkv * 256;
    a->ws_bytes = workspace_bytes(rp);
    a->ws = take(a->ws_bytes);
    a->scores = reinterpret_cast<float*>(take((size_t)(n_sig > 0 ? n_sig : 1) * rp.L_d * 4));
    a->idx_in = reinterpret_cast<int32_t*>(take((size_t)rp.L_d * 4));
    a->idx_out = reinterpret_cast<int32_t*>(take((size_t)rp.L_d * 4));
    a->q_fresh = take(qrow * rp.N);
    a->k_fresh = take(kvrow * rp.N);
    a->v_fresh = take(kvrow * rp.N);
    a->kv_k = take(kvrow * rp.N);
    a->kv_v = take(kvrow * rp.N);
    a->q_pack = take(qrow * rp.k);
    a->k_pack = take(kvrow * rp.k);
    a->v_pack = take(kvrow * rp.k);
    a->hidden = take(qrow * (rp.fuse_mode == 1 ? rp.N : rp.k + rp.L_q));
    a->total = off;
}
constexpr int kArenaSignalRows = 8;   // arena is sized for up to this many signal rows
// From this many important tokens on the host-buffer layer skips the packed copy of the Q rows (step 2 reads
// them in place): measured -2 % layer time at k = 41780, +-1 % at k = 6554, +10 % at k = 922.
constexpr int kQInPlaceMinK = 16384;

// True (and *dev set) when `h` is pinned host memory that kernels on the current device can address.
bool mapped_host_pointer(const void* h, const void** dev) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, h) != cudaSuccess) { (void)cudaGetLastError(); return false; }
    if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) return false;
    *dev = attr.devicePointer;
    return true;
}
}  // namespace

size_t daf_layer_host_arena_bytes(const daf_params* p) {
    ResolvedParams rp;
    if (resolve_params(p, &rp) != DAF_OK) return 0;
    Arena a;
    carve_arena(rp, kArenaSignalRows, nullptr, &a);
    return a.total;
}


int daf_layer_host_begin(const daf_params* p, const float* h_scores, int32_t n_sig, const int32_t* h_idx_in,
                         const void* h_q_fresh, const void* h_k_fresh, const void* h_v_fresh,
                         void* h_kv_k, void* h_kv_v, int32_t copy_back_kv,
                         void* h_hidden, int32_t* h_idx_out,
                         void* arena, size_t arena_bytes, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    if (h_scores != nullptr && (n_sig < 1 || n_sig > kArenaSignalRows)) return DAF_ERR_INVALID_ARG;
    if (arena == nullptr || !aligned16(arena)) return DAF_ERR_WORKSPACE;
    Arena a;
    carve_arena(rp, kArenaSignalRows, reinterpret_cast<char*>(arena), &a);
    if (arena_bytes < a.total) return DAF_ERR_WORKSPACE;
    if (rp.k + rp.L_q == 0) return DAF_OK;
    if (!h_q_fresh || !h_k_fresh || !h_v_fresh || !h_kv_k || !h_kv_v || !h_hidden) return DAF_ERR_INVALID_ARG;
    if (rp.k > 0 && !h_scores && !h_idx_in) return DAF_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t qrow = (size_t)rp.Hq * 256, kvrow = (size_t)rp.Hkv * 256;
    DAF_CUDA_TRY(cudaMemsetAsync(a.ws, 0, kStatusBytes, st));
    if (h_scores) DAF_CUDA_TRY(cudaMemcpyAsync(a.scores, h_scores, (size_t)n_sig * rp.L_d * 4, cudaMemcpyHostToDevice, st));
    else if (rp.k > 0) DAF_CUDA_TRY(cudaMemcpyAsync(a.idx_in, h_idx_in, (size_t)rp.k * 4, cudaMemcpyHostToDevice, st));
    // Of the fresh tensors the layer touches only the rows of the important tokens and of the question.  When the
    // three host tensors are pinned memory that the device can address, the gather / cache-update kernel reads those
    // rows straight from the host (k + L_q rows instead of N cross the link) and only the question's Q rows, which
    // the attention kernel reads through a tensor map, are copied; otherwise the tensors are copied whole.
    RowSource rows = {nullptr, nullptr, nullptr};
    const bool in_place_rows = rp.k > 0 && mapped_host_pointer(h_q_fresh, &rows.q) && mapped_host_pointer(h_k_fresh, &rows.k) &&
                               mapped_host_pointer(h_v_fresh, &rows.v);
    if (in_place_rows) {
        if (rp.L_q > 0)
            DAF_CUDA_TRY(cudaMemcpyAsync(reinterpret_cast<char*>(a.q_fresh) + qrow * rp.L_d,
                                         reinterpret_cast<const char*>(h_q_fresh) + qrow * rp.L_d, qrow * rp.L_q,
                                         cudaMemcpyHostToDevice, st));
    } else {
        DAF_CUDA_TRY(cudaMemcpyAsync(a.q_fresh, h_q_fresh, qrow * rp.N, cudaMemcpyHostToDevice, st));
        DAF_CUDA_TRY(cudaMemcpyAsync(a.k_fresh, h_k_fresh, kvrow * rp.N, cudaMemcpyHostToDevice, st));
        DAF_CUDA_TRY(cudaMemcpyAsync(a.v_fresh, h_v_fresh, kvrow * rp.N, cudaMemcpyHostToDevice, st));
    }
    // only the document rows of the cache carry information on entry
    DAF_CUDA_TRY(cudaMemcpyAsync(a.kv_k, h_kv_k, kvrow * rp.L_d, cudaMemcpyHostToDevice, st));
    DAF_CUDA_TRY(cudaMemcpyAsync(a.kv_v, h_kv_v, kvrow * rp.L_d, cudaMemcpyHostToDevice, st));
    // (rows read from the host: always with packed copies on the device, the attention kernel must not go to the host)
    void* qp = (!in_place_rows && rp.k >= kQInPlaceMinK && rp.L_q > 0) ? nullptr : a.q_pack;
    if (int rc = layer_impl(p, nullptr, h_scores ? a.scores : nullptr, n_sig, h_scores ? nullptr : a.idx_in, a.q_fresh, a.k_fresh,
                            a.v_fresh, a.kv_k, a.kv_v, a.idx_out, qp, a.k_pack, a.v_pack, a.hidden, nullptr, a.ws, a.ws_bytes, stream,
                            in_place_rows ? &rows : nullptr)) return rc;
    const size_t hidden_rows = rp.fuse_mode == 1 ? rp.N : rp.k + rp.L_q;
    DAF_CUDA_TRY(cudaMemcpyAsync(h_hidden, a.hidden, qrow * hidden_rows, cudaMemcpyDeviceToHost, st));
    if (h_idx_out && rp.k > 0) DAF_CUDA_TRY(cudaMemcpyAsync(h_idx_out, a.idx_out, (size_t)rp.k * 4, cudaMemcpyDeviceToHost, st));
    if (copy_back_kv) {
        DAF_CUDA_TRY(cudaMemcpyAsync(h_kv_k, a.kv_k, kvrow * rp.N, cudaMemcpyDeviceToHost, st));
        DAF_CUDA_TRY(cudaMemcpyAsync(h_kv_v, a.kv_v, kvrow * rp.N, cudaMemcpyDeviceToHost, st));
    }
    return DAF_OK;
}

int daf_layer_host_end(const daf_params* p, void* arena, size_t arena_bytes, void* stream) {
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    if (arena == nullptr || !aligned16(arena)) return DAF_ERR_WORKSPACE;
    Arena a;
    carve_arena(rp, kArenaSignalRows, reinterpret_cast<char*>(arena), &a);
    if (arena_bytes < a.total) return DAF_ERR_WORKSPACE;
    DAF_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    if (rp.k + rp.L_q == 0) return DAF_OK;
    DeviceStatus hs;
    DAF_CUDA_TRY(cudaMemcpy(&hs, a.ws, sizeof(hs), cudaMemcpyDeviceToHost));
    return hs.code;
}

int daf_layer_host(const daf_params* p, const float* h_scores, int32_t n_sig, const int32_t* h_idx_in,
                   const void* h_q_fresh, const void* h_k_fresh, const void* h_v_fresh,
                   void* h_kv_k, void* h_kv_v, int32_t copy_back_kv,
                   void* h_hidden, int32_t* h_idx_out,
                   void* arena, size_t arena_bytes, void* stream) {
    if (int rc = daf_layer_host_begin(p, h_scores, n_sig, h_idx_in, h_q_fresh, h_k_fresh, h_v_fresh, h_kv_k, h_kv_v,
                                      copy_back_kv, h_hidden, h_idx_out, arena, arena_bytes, stream)) return rc;
    return daf_layer_host_end(p, arena, arena_bytes, stream);
}

int daf_workspace_init(void* workspace, size_t workspace_bytes_, void* stream) {
    if (workspace == nullptr || workspace_bytes_ < kStatusBytes) return DAF_ERR_WORKSPACE;
    DAF_CUDA_TRY(cudaMemsetAsync(workspace, 0, kStatusBytes, (cudaStream_t)stream));
    return DAF_OK;
}

int daf_poll_status(void* workspace, void* stream) {
    if (workspace == nullptr) return DAF_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    DeviceStatus hs;
    DAF_CUDA_TRY(cudaMemcpyAsync(&hs, workspace, sizeof(hs), cudaMemcpyDeviceToHost, st));
    DAF_CUDA_TRY(cudaStreamSynchronize(st));
    if (hs.code != 0) {
        DAF_CUDA_TRY(cudaMemsetAsync(workspace, 0, sizeof(hs), st));
        DAF_CUDA_TRY(cudaStreamSynchronize(st));
    }
    return hs.code;
}

int daf_selftest_bounded_wait(void* workspace, size_t workspace_bytes_, int32_t limit_ms, void* stream) {
    if (workspace == nullptr || workspace_bytes_ < kStatusBytes) return DAF_ERR_WORKSPACE;
    if (limit_ms < 1 || limit_ms > 1000) return DAF_ERR_INVALID_ARG;
    return launch_bounded_wait_selftest(reinterpret_cast<DeviceStatus*>(workspace), limit_ms, (cudaStream_t)stream);
}

const char* daf_strerror(int status) {
    switch (status) {
        case DAF_OK: return "ok";
        case DAF_ERR_INVALID_ARG: return "invalid argument";
        case DAF_ERR_UNSUPPORTED: return "unsupported shape (head_dim must be 128, n_q_heads a multiple of n_kv_heads)";
        case DAF_ERR_ALIGNMENT: return "pointer or stride not 16-byte aligned";
        case DAF_ERR_WORKSPACE: return "workspace missing or too small";
        case DAF_ERR_CUDA: return "CUDA call failed (see daf_last_cuda_error)";
        case DAF_ERR_TIMEOUT: return "device-side bounded wait ran out";
        case DAF_ERR_BOUNDS: return "device-side index out of range";
        default: return "unknown status";
    }
}

int daf_last_cuda_error(void) { return g_last_cuda_error; }

int64_t daf_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
