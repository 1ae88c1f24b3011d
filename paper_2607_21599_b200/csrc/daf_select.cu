// Step 1 of the DAF layer (Methods, item 1 "selection" and "gather"; item 2
// "hybrid KV cache") and the stand-alone form of step 4 (item 3 "state fusion").
//
// These steps move bytes and rank 32-bit keys; they are bound by HBM bandwidth
// and launch latency, not by arithmetic, so they are plain coalesced 16-byte
// kernels with no tensor-core work.
#include "daf_common.cuh"

namespace daf {

// ------------------------------------------------------------------ selection
// One CTA ranks all L_d aggregated scores: an 8-bit-per-pass radix select finds
// the key of the k-th largest score, then an ordered compaction emits the
// selected positions in ascending order.  Ties at the threshold are broken by
// position (lower first), which makes the result unique.

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelSmemKeys = 40960;  // keys kept in shared memory up to this L_d, in global scratch beyond

// Monotone map fp32 -> uint32: larger score <=> larger key; -0 == +0; NaN -> 0 (ranks lowest).
__device__ __forceinline__ uint32_t score_key(float s) {
    uint32_t b = __float_as_uint(s);
    if ((b & 0x7FFFFFFFu) > 0x7F800000u) return 0u;   // NaN
    if (b == 0x80000000u) b = 0u;                     // -0 -> +0
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__global__ void __launch_bounds__(kSelThreads, 1)
select_topk_kernel(const float* __restrict__ scores, int n_sig, int L_d, int k,
                   uint32_t* __restrict__ gkeys, int32_t* __restrict__ idx_out) {
    extern __shared__ __align__(16) unsigned char sel_smem[];
    uint32_t* hist = reinterpret_cast<uint32_t*>(sel_smem);              // [kSelWarps][256]
    uint32_t* total = hist + kSelWarps * 256;                             // [256]
    uint32_t* scan_gt = total + 256;                                      // [kSelWarps]
    uint32_t* scan_eq = scan_gt + kSelWarps;                              // [kSelWarps]
    uint32_t* sh = scan_eq + kSelWarps;                                   // [4]: prefix, k_rem
    uint32_t* skeys = sh + 4;
    uint32_t* keys = (L_d <= kSelSmemKeys) ? skeys : gkeys;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // aggregate the signal rows in ascending row order (fp32 adds, no fusing) and build keys
    for (int i = tid; i < L_d; i += kSelThreads) {
        float acc = scores[i];
        for (int l = 1; l < n_sig; ++l) acc = __fadd_rn(acc, scores[(size_t)l * L_d + i]);
        keys[i] = score_key(acc);
    }
    if (tid == 0) { sh[0] = 0u; sh[1] = (uint32_t)k; }
    __syncthreads();

    uint32_t prefix = 0u, mask = 0u;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < kSelWarps * 256; i += kSelThreads) hist[i] = 0u;
        __syncthreads();
        const int n_round = (L_d + kSelThreads - 1) / kSelThreads * kSelThreads;
        for (int i = tid; i < n_round; i += kSelThreads) {
            bool in = false;
            uint32_t bin = 0xFFFFFFFFu;
            if (i < L_d) {
                const uint32_t key = keys[i];
                in = (key & mask) == prefix;
                if (in) bin = (key >> shift) & 0xFFu;
            }
            // warp-aggregated histogram update: one atomic per distinct bin in the warp
            const uint32_t peers = __match_any_sync(0xFFFFFFFFu, bin);
            if (in && (int)(__ffs(peers) - 1) == lane) atomicAdd(&hist[warp * 256 + bin], (uint32_t)__popc(peers));
        }
        __syncthreads();
        if (tid < 256) {
            uint32_t s = 0;
            for (int w = 0; w < kSelWarps; ++w) s += hist[w * 256 + tid];
            total[tid] = s;
        }
        __syncthreads();
        if (warp == 0) {
            // lane l owns bins [8*(31-l), 8*(31-l)+7]; lane 0 holds the highest bins
            const int base = 8 * (31 - lane);
            uint32_t s = 0;
            for (int b = 0; b < 8; ++b) s += total[base + b];
            uint32_t incl = s;
            for (int o = 1; o < 32; o <<= 1) {
                uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += t;
            }
            const uint32_t above = incl - s;
            const uint32_t k_rem = sh[1];
            if (k_rem > above && k_rem <= incl) {
                uint32_t a = above;
                for (int b = 7; b >= 0; --b) {
                    const uint32_t c = total[base + b];
                    if (k_rem <= a + c) {
                        sh[0] = prefix | ((uint32_t)(base + b) << shift);
                        sh[1] = k_rem - a;
                        break;
                    }
                    a += c;
                }
            }
        }
        __syncthreads();
        prefix = sh[0];
        mask |= 0xFFu << shift;
    }
    const uint32_t thr = prefix;       // key of the k-th largest score
    const uint32_t need_eq = sh[1];    // how many keys equal to thr are taken (lowest positions first)

    // ordered compaction: thread t owns the contiguous positions [t*E, (t+1)*E)
    const int E = (L_d + kSelThreads - 1) / kSelThreads;
    const int lo = min(L_d, tid * E), hi = min(L_d, lo + E);
    uint32_t n_gt = 0, n_eq = 0;
    for (int i = lo; i < hi; ++i) {
        const uint32_t key = keys[i];
        n_gt += key > thr;
        n_eq += key == thr;
    }
    uint32_t in_gt = n_gt, in_eq = n_eq;
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t a = __shfl_up_sync(0xFFFFFFFFu, in_gt, o), b = __shfl_up_sync(0xFFFFFFFFu, in_eq, o);
        if (lane >= o) { in_gt += a; in_eq += b; }
    }
    if (lane == 31) { scan_gt[warp] = in_gt; scan_eq[warp] = in_eq; }
    __syncthreads();
    if (warp == 0) {
        uint32_t a = scan_gt[lane], b = scan_eq[lane];
        uint32_t ia = a, ib = b;
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t x = __shfl_up_sync(0xFFFFFFFFu, ia, o), y = __shfl_up_sync(0xFFFFFFFFu, ib, o);
            if (lane >= o) { ia += x; ib += y; }
        }
        scan_gt[lane] = ia - a;
        scan_eq[lane] = ib - b;
    }
    __syncthreads();
    uint32_t gt_before = scan_gt[warp] + in_gt - n_gt;
    uint32_t eq_before = scan_eq[warp] + in_eq - n_eq;
    if (k > 0) {
        uint32_t pos = gt_before + min(eq_before, need_eq);
        for (int i = lo; i < hi; ++i) {
            const uint32_t key = keys[i];
            bool take = key > thr;
            if (key == thr) { take = eq_before < need_eq; ++eq_before; }
            if (take) idx_out[pos++] = i;
        }
    }
}

// --------------------------------------------------- gather + hybrid KV update
// One CTA per row.  Rows 0..k-1 are the important tokens: their fresh Q/K/V rows
// go to the packed buffers and (K/V) into the cache rows at their positions.
// Rows k..k+L_q-1 are the question tokens: fresh K/V rows are appended to the cache.
constexpr int kRowThreads = 192;

struct GatherArgs {
    const int4* q_fresh; const int4* k_fresh; const int4* v_fresh;
    int4* kv_k; int4* kv_v;
    int4* q_pack; int4* k_pack; int4* v_pack;
    const int32_t* idx;       // positions to gather (idx_in, or idx_out written by the select kernel)
    int32_t* idx_copy;        // when non-null, also receives idx (the idx_in path)
    int k, L_d, L_q, cq, ckv; // cq/ckv: 16-byte chunks per Q row / per K (or V) row
    int overwrite;
    DeviceStatus* status;
};

__global__ void __launch_bounds__(kRowThreads)
gather_update_kernel(const GatherArgs a) {
    const int row = blockIdx.x;
    const int per_row = a.cq + 2 * a.ckv;
    if (row < a.k) {
        const int p = a.idx[row];
        if (a.idx_copy != nullptr && threadIdx.x == 0) a.idx_copy[row] = p;
        if (p < 0 || p >= a.L_d) {
            if (threadIdx.x == 0) report_status(a.status, DAF_ERR_BOUNDS, 1, p);
            return;
        }
        const size_t qsrc = (size_t)p * a.cq, qdst = (size_t)row * a.cq;
        const size_t ksrc = (size_t)p * a.ckv, kdst = (size_t)row * a.ckv;
        for (int c = threadIdx.x; c < per_row; c += kRowThreads) {
            if (c < a.cq) {
                a.q_pack[qdst + c] = __ldg(a.q_fresh + qsrc + c);
            } else if (c < a.cq + a.ckv) {
                const int cc = c - a.cq;
                const int4 v = __ldg(a.k_fresh + ksrc + cc);
                a.k_pack[kdst + cc] = v;
                if (a.overwrite) a.kv_k[ksrc + cc] = v;
            } else {
                const int cc = c - a.cq - a.ckv;
                const int4 v = __ldg(a.v_fresh + ksrc + cc);
                a.v_pack[kdst + cc] = v;
                if (a.overwrite) a.kv_v[ksrc + cc] = v;
            }
        }
    } else {
        const size_t off = (size_t)(a.L_d + (row - a.k)) * a.ckv;
        for (int c = threadIdx.x; c < 2 * a.ckv; c += kRowThreads) {
            if (c < a.ckv) a.kv_k[off + c] = __ldg(a.k_fresh + off + c);
            else a.kv_v[off + c - a.ckv] = __ldg(a.v_fresh + off + c - a.ckv);
        }
    }
}

// ------------------------------------------------------------- state fusion
struct FuseArgs {
    const int4* o_imp; const int4* o_q; int4* hidden;
    const int32_t* idx; int32_t* row_pos;
    int k, L_d, L_q, cq, mode;
    DeviceStatus* status;
};

__global__ void __launch_bounds__(kRowThreads)
fuse_rows_kernel(const FuseArgs a) {
    const int row = blockIdx.x;
    int pos;
    const int4* src;
    if (row < a.k) { pos = a.idx[row]; src = a.o_imp + (size_t)row * a.cq; }
    else { pos = a.L_d + (row - a.k); src = a.o_q + (size_t)(row - a.k) * a.cq; }
    if (a.row_pos != nullptr && threadIdx.x == 0) a.row_pos[row] = pos;
    if (a.hidden == nullptr) return;
    if (pos < 0 || pos >= a.L_d + a.L_q) return;
    int4* dst = a.hidden + (size_t)(a.mode == 0 ? row : pos) * a.cq;
    for (int c = threadIdx.x; c < a.cq; c += kRowThreads) dst[c] = __ldg(src + c);
}

// ----------------------------------------------------------------- host side
size_t select_scratch_bytes(int L_d) {
    return L_d > kSelSmemKeys ? ((size_t)L_d * sizeof(uint32_t) + 255) / 256 * 256 : 0;
}

static size_t select_smem_bytes(int L_d) {
    size_t fixed = (size_t)(kSelWarps * 256 + 256 + 2 * kSelWarps + 4) * sizeof(uint32_t);
    return fixed + (L_d <= kSelSmemKeys ? (size_t)L_d * sizeof(uint32_t) : 0);
}

int launch_select(const ResolvedParams& rp, const float* scores, int n_sig, const int32_t* idx_in,
                  const void* q_fresh, const void* k_fresh, const void* v_fresh, void* kv_k, void* kv_v,
                  int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack,
                  DeviceStatus* status, void* scratch, cudaStream_t stream) {
    const int32_t* idx_src = idx_in;
    if (scores != nullptr && rp.L_d > 0) {
        static bool attr_set = false;
        const size_t smem = select_smem_bytes(rp.L_d);
        if (!attr_set) {
            cudaError_t e = cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)select_smem_bytes(kSelSmemKeys));
            if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
            attr_set = true;
        }
        select_topk_kernel<<<1, kSelThreads, smem, stream>>>(scores, n_sig, rp.L_d, rp.k,
                                                            reinterpret_cast<uint32_t*>(scratch), idx_out);
        count_launch();
        if (int rc = check_launch()) return rc;
        idx_src = idx_out;
    }
    const int rows = rp.k + rp.L_q;
    if (rows > 0) {
        GatherArgs a;
        a.q_fresh = reinterpret_cast<const int4*>(q_fresh);
        a.k_fresh = reinterpret_cast<const int4*>(k_fresh);
        a.v_fresh = reinterpret_cast<const int4*>(v_fresh);
        a.kv_k = reinterpret_cast<int4*>(kv_k);
        a.kv_v = reinterpret_cast<int4*>(kv_v);
        a.q_pack = reinterpret_cast<int4*>(q_pack);
        a.k_pack = reinterpret_cast<int4*>(k_pack);
        a.v_pack = reinterpret_cast<int4*>(v_pack);
        a.idx = idx_src;
        a.idx_copy = (idx_src == idx_in && idx_out != nullptr && idx_out != idx_in) ? idx_out : nullptr;
        a.k = rp.k; a.L_d = rp.L_d; a.L_q = rp.L_q;
        a.cq = rp.Hq * 16; a.ckv = rp.Hkv * 16;
        a.overwrite = rp.overwrite;
        a.status = status;
        gather_update_kernel<<<rows, kRowThreads, 0, stream>>>(a);
        count_launch();
        if (int rc = check_launch()) return rc;
    }
    return DAF_OK;
}

int launch_fuse(const ResolvedParams& rp, const int32_t* idx, const void* o_imp, const void* o_q, void* hidden,
                int32_t* row_pos_out, cudaStream_t stream) {
    const int rows = rp.k + rp.L_q;
    if (rows == 0) return DAF_OK;
    FuseArgs a;
    a.o_imp = reinterpret_cast<const int4*>(o_imp);
    a.o_q = reinterpret_cast<const int4*>(o_q);
    a.hidden = reinterpret_cast<int4*>(hidden);
    a.idx = idx; a.row_pos = row_pos_out;
    a.k = rp.k; a.L_d = rp.L_d; a.L_q = rp.L_q; a.cq = rp.Hq * 16; a.mode = rp.fuse_mode;
    a.status = nullptr;
    fuse_rows_kernel<<<rows, kRowThreads, 0, stream>>>(a);
    count_launch();
    return check_launch();
}

}  // namespace daf
