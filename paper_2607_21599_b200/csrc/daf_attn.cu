// Steps 2 and 3 of the DAF layer and the full-recompute comparison path: dense
// softmax attention with a causal limit (Methods, items 1 and 2; complexity
// analysis: the r^2 L_d^2 and L_q (L_d + L_q) terms).
//
// One kernel (attn_fwd_kernel, described where it is defined) serves all of them;
// a second one merges the partial results of launches that cut the key axis into
// ranges.  A launch runs one attention problem, or -- for a DAF layer -- the
// important-token stage and the question stage together from one list of work
// items.
#include <math.h>
#include <string.h>

#include <atomic>
#include <functional>
#include <map>
#include <mutex>
#include <queue>
#include <vector>

#include "daf_common.cuh"

namespace daf {

constexpr int kBlockM = 128;            // rows per query tile
constexpr int kBlockN = 128;            // keys per KV tile
constexpr int kD = 128;                 // head_dim
constexpr int kTileBytes = kBlockN * kD * 2;      // 32 KB: one Q tile, or K (or V) of 128 keys
constexpr int kHalfBytes = kTileBytes / 2;        // one 64-column half (128-byte rows)
constexpr int kMaxSplits = 32;
constexpr int kNumSMsDefault = 148;    // B200; the planners ask the device (num_sms below)
constexpr float kRescaleThreshold = 8.0f;   // in log2 units: keep a stale row maximum up to 2^8

// One attention problem and how it is cut into work items.
struct SegArgs {
    int n_q;            // query tokens
    int n_kv;           // key rows
    int Hq, G;          // query heads; group size Hq / Hkv
    int Gp;             // query heads per tile (1 or G)
    int Tt;             // tokens per tile = 128 / Gp
    int n_tb;           // token blocks = ceil(n_q / Tt)
    int causal_off;     // token t sees keys <= t + causal_off ...
    const int32_t* q_pos; // ... or, when given, keys <= q_pos[t] (ascending positions of the query tokens)
    // Query rows read in place instead of from a packed copy (Gp == 1 only): query token t is row q_idx[t]
    // of q_src, a [q_src_rows, Hq, 128] tensor.  q_idx == nullptr: the Q tensor map covers packed rows.
    const __nv_bfloat16* q_src;
    const int32_t* q_idx;
    int q_src_rows;
    // Likewise the keys: key j is row kv_idx[j] of k_src / v_src, [kv_src_rows, kv_heads, 128] tensors.
    // k_src == nullptr: the K and V tensor maps cover packed rows.
    const __nv_bfloat16* k_src;
    const __nv_bfloat16* v_src;
    const int32_t* kv_idx;
    int kv_src_rows, kv_heads;
    // Work items.  A CTA owns one token block (a unit).  Either every unit is cut into the same n_splits
    // KV ranges of tiles_per_split tiles (chunk == 0), or -- packed causal attention only, where unit u
    // sees min(u + 1, n_tb) tiles -- units [g chunk, (g + 1) chunk) are cut into g + 1 balanced ranges
    // each, so that no item walks more than about `chunk` tiles.
    int head_blocks, n_units;
    int n_splits, tiles_per_split;
    int chunk, n_slots;    // n_slots: number of (unit, range) pairs = partial-result slots
    int n_items;           // head_blocks * (n_units * n_splits  or  n_slots)
    float scale;        // softmax scale
    float scale_log2;   // scale * log2(e)
    __nv_bfloat16* out; long long out_row_stride;  // elements
    const int32_t* dst_rows;
    int out_tiled;      // final rows leave by one tiled bulk store per tile (rows in token order, no dst_rows)
    float* lse;         // [Hq, n_q] or null
    float* part_o;      // partial results, fp32, normalised per range: [slot rows][Hq][128]
    float* part_lse;    // [slot rows][Hq]
};

// A launch runs one problem on a 3-D grid (head block, unit, split), or two problems from one list of
// items on a 1-D grid (joint): the items of seg[1] first, then those of seg[0], heaviest units first.
struct AttnArgs {
    SegArgs seg[2];
    int joint;
    DeviceStatus* status;
};

#ifdef DAF_TRACE
// Debug build only (-DDAF_TRACE): per-CTA time stamps for latency studies.
__device__ unsigned long long g_trace[8 * 65536];
DAF_KT_TABLE;
DAF_KT_READER(daf_dbg_kt_attn)
// per-CTA clock totals of the first softmax thread: total, wait S, softmax, wait P V + rescale, epilogue, sub-steps
__device__ long long g_laps[8 * 65536];
extern "C" int daf_dbg_read_laps(void* host, size_t bytes) {
    return (int)cudaMemcpyFromSymbol(host, g_laps, bytes < sizeof(g_laps) ? bytes : sizeof(g_laps));
}
#define DAF_LAP_DECL long long lap_s = 0, lap_soft = 0, lap_pv = 0, lap_t = clock64(); const long long lap_begin = lap_t
#define DAF_LAP(acc) do { const long long now_ = clock64(); acc += now_ - lap_t; lap_t = now_; } while (0)
#define DAF_STAMP(slot)                                                                         \
    do {                                                                                        \
        const unsigned cta_ = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);   \
        if (cta_ < 65536u) g_trace[8 * cta_ + (slot)] = global_ns();                            \
    } while (0)
#else
#define DAF_STAMP(slot) do {} while (0)
#define DAF_LAP_DECL do {} while (0)
#define DAF_LAP(acc) do {} while (0)
#endif

// One online-softmax step of one query row (one thread) over NCH * 32 keys starting at `key0` (the kernel
// uses NCH = 2, a 64-key sub-step): reads the row's logits from tensor memory, writes P = exp(s - m) as bf16 over the first half of the same columns,
// keeps the running maximum m and sum l.  Returns the factor the row of O has to be multiplied by (1
// unless the maximum grew past the lazy threshold).  `limit` is the last key the row may see;
// c = softmax scale * log2(e).
template <int NCH>
__device__ __forceinline__ float softmax_core(uint32_t s_addr, int key0, int limit, float c, float& m, float& l) {
    constexpr int H = NCH / 2;
    // the logits are fetched in two halves so that the row maximum of the first half is computed
    // while the second half is still on its way from tensor memory
    uint32_t sr[NCH][32];
#pragma unroll
    for (int i = 0; i < H; ++i) tmem_ld32(s_addr + (uint32_t)(32 * i), sr[i]);
    tc_wait_ld();
#pragma unroll
    for (int i = H; i < NCH; ++i) tmem_ld32(s_addr + (uint32_t)(32 * i), sr[i]);
    const bool need_mask = key0 + NCH * 32 - 1 > limit;
    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        if (half == 1) tc_wait_ld();
        if (need_mask) {
#pragma unroll
            for (int cchunk = H * half; cchunk < H * half + H; ++cchunk)
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (key0 + cchunk * 32 + i > limit) sr[cchunk][i] = 0xFF800000u;  // -inf
        }
#pragma unroll
        for (int cchunk = H * half; cchunk < H * half + H; ++cchunk)
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
                // four independent chains of 3-input maxima
                mx[0] = fmax3(mx[0], __uint_as_float(sr[cchunk][i + 0]), __uint_as_float(sr[cchunk][i + 1]));
                mx[1] = fmax3(mx[1], __uint_as_float(sr[cchunk][i + 2]), __uint_as_float(sr[cchunk][i + 3]));
                mx[2] = fmax3(mx[2], __uint_as_float(sr[cchunk][i + 4]), __uint_as_float(sr[cchunk][i + 5]));
                mx[3] = fmax3(mx[3], __uint_as_float(sr[cchunk][i + 6]), __uint_as_float(sr[cchunk][i + 7]));
            }
    }
    const float tmax = fmax3(mx[0], mx[1], fmaxf(mx[2], mx[3]));
    float m_new = fmaxf(m, tmax);
    // keep a slightly stale maximum: rescaling O is skipped while the growth stays below 2^8
    if (m != -INFINITY && (m_new - m) * c <= kRescaleThreshold) m_new = m;
    const float m_used = (m_new == -INFINITY) ? 0.f : m_new;
    const float alpha = (m == -INFINITY) ? 1.f : fast_exp2((m - m_new) * c);
    const float mc = m_used * c;
    // p = 2^(s*c - m*c): packed two-wide FMA and adds, exponentials on the special-function unit
    const uint64_t c2 = pack_f32x2(c, c), nmc2 = pack_f32x2(-mc, -mc);
    uint64_t acc2[4] = {0ull, 0ull, 0ull, 0ull};
    uint32_t pr[H][32];
#pragma unroll
    for (int cchunk = 0; cchunk < NCH; ++cchunk)
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
            const uint64_t x2 = ffma2(pack_f32x2(__uint_as_float(sr[cchunk][i]), __uint_as_float(sr[cchunk][i + 1])), c2, nmc2);
            const float p0 = fast_exp2(f32x2_lo(x2));
            const float p1 = fast_exp2(f32x2_hi(x2));
            acc2[(i >> 1) & 3] = fadd2(acc2[(i >> 1) & 3], pack_f32x2(p0, p1));
            pr[cchunk >> 1][(cchunk & 1) * 16 + (i >> 1)] = pack_bf16(p0, p1);
        }
    const uint64_t acc01 = fadd2(fadd2(acc2[0], acc2[1]), fadd2(acc2[2], acc2[3]));
    const float rowsum = f32x2_lo(acc01) + f32x2_hi(acc01);
    l = l * alpha + rowsum;
    m = m_new;
    // P (bf16, two keys per 32-bit column) overlays the first half of the columns of S
#pragma unroll
    for (int i = 0; i < H; ++i) tmem_st32(s_addr + (uint32_t)(32 * i), pr[i]);
    return alpha;
}

// Multiplies this thread's row of O (128 fp32 columns in tensor memory) by alpha.  O must be quiescent.
__device__ __forceinline__ void rescale_o(uint32_t o_addr, float alpha) {
#pragma unroll
    for (int cchunk = 0; cchunk < 4; ++cchunk) {
        uint32_t orr[32];
        tmem_ld32(o_addr + (uint32_t)(cchunk * 32), orr);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * alpha);
        tmem_st32(o_addr + (uint32_t)(cchunk * 32), orr);
    }
}

// Picks a field of the problem a CTA works on (seg_id is uniform across the CTA).
#define DAF_SEG(field) (seg_id ? args.seg[1].field : args.seg[0].field)

// What one CTA works on: the problem's geometry and the CTA's item (one token block of one head
// block, and a range of key tiles).
struct CtaWork {
    int n_q, n_kv, G, Gp, Tt, n_tb, causal_off;
    const int32_t* q_pos;
    float scale_log2;
    int seg_id, hb, unit, j_begin, j_end, item_splits, tok_base;
    long long part_row0;      // the item's first row in the partial-result arrays, in tokens
};

__device__ __forceinline__ void decode_work(const AttnArgs& args, CtaWork& a) {
    // ---- which item is this CTA's (uniform across the CTA)
    int seg_id = 0, item = (int)blockIdx.x;
    if (args.joint) {
        if (item < args.seg[1].n_items) seg_id = 1;
        else item -= args.seg[1].n_items;
    }
    a.n_q = DAF_SEG(n_q); a.n_kv = DAF_SEG(n_kv); a.G = DAF_SEG(G); a.Gp = DAF_SEG(Gp); a.Tt = DAF_SEG(Tt);
    a.n_tb = DAF_SEG(n_tb); a.causal_off = DAF_SEG(causal_off); a.q_pos = DAF_SEG(q_pos); a.scale_log2 = DAF_SEG(scale_log2);

    int hb, unit, j_begin, j_end, item_splits, tok_base;
    long long part_row0;      // this item's first row in the partial-result arrays, in tokens
    if (!args.joint || DAF_SEG(chunk) == 0) {
        int split;
        if (!args.joint) {
            // blocks are dispatched x-fastest: all head blocks of the heaviest (last) unit go first
            hb = (int)blockIdx.x; unit = (int)gridDim.y - 1 - (int)blockIdx.y; split = (int)blockIdx.z;
        } else {
            const int n_hb = DAF_SEG(head_blocks), n_units = DAF_SEG(n_units);
            hb = item % n_hb;
            const int rest = item / n_hb;
            unit = n_units - 1 - rest % n_units;
            split = rest / n_units;
        }
        const int tps = DAF_SEG(tiles_per_split);
        j_begin = split * tps;
        j_end = j_begin + tps;
        item_splits = DAF_SEG(n_splits);
        part_row0 = (long long)split * a.n_q;
        tok_base = 0;
    } else {
        // packed causal attention cut into balanced ranges: slot numbers ascend with the unit, the
        // grid walks them from the top so that the longest items start first
        const int n_hb = DAF_SEG(head_blocks), chunk = DAF_SEG(chunk);
        hb = item % n_hb;
        const int slot = DAF_SEG(n_slots) - 1 - item / n_hb;
        int g = (int)((sqrtf(1.f + 8.f * (float)slot / (float)chunk) - 1.f) * 0.5f);
        while (chunk * (g + 1) * (g + 2) / 2 <= slot) ++g;
        while (g > 0 && chunk * g * (g + 1) / 2 > slot) --g;
        const int rem = slot - chunk * g * (g + 1) / 2;
        unit = g * chunk + rem / (g + 1);
        const int range = rem % (g + 1);
        const int n_tiles = min(unit + 1, a.n_tb);
        j_begin = range * n_tiles / (g + 1);
        j_end = (range + 1) * n_tiles / (g + 1);
        item_splits = g + 1;
        part_row0 = (long long)slot * kBlockM;
        tok_base = unit * kBlockM;
    }
    a.seg_id = seg_id; a.hb = hb; a.unit = unit; a.j_begin = j_begin; a.j_end = j_end;
    a.item_splits = item_splits; a.tok_base = tok_base; a.part_row0 = part_row0;
}

// Final step of a tile: the warp's 32 rows of O (fp32 in tensor memory at o_addr, this thread's row
// unnormalised with running maximum m and sum l) leave as bf16 output rows, or -- for an item that
// covers only part of the keys -- as fp32 partial rows with their log-sum-exp.
__device__ __forceinline__ void write_rows(const AttnArgs& args, const CtaWork& a, int t0, bool has_keys, bool row_valid,
                                           bool row_valid_tile, int tok, int head, int h0, unsigned char* q_tile,
                                           const CUtensorMap* tmap_o, uint64_t* rows_parked, volatile int* abort_flag,
                                           uint32_t o_addr, int quad, int lane, float m, float l) {
    unsigned char* const stage = q_tile + (size_t)quad * 32 * 256;   // this warp's part of the dead Q tile
    const int seg_id = a.seg_id;
    // the fields only the epilogue needs are picked here, not held in registers through the loop
    struct { int n_q, Gp, Tt, Hq; __nv_bfloat16* out; long long out_row_stride; const int32_t* dst_rows;
             float* lse; float* part_o; float* part_lse; } e;
    e.n_q = a.n_q; e.Gp = a.Gp; e.Tt = a.Tt; e.Hq = DAF_SEG(Hq);
    e.out = DAF_SEG(out); e.out_row_stride = DAF_SEG(out_row_stride); e.dst_rows = DAF_SEG(dst_rows);
    e.lse = DAF_SEG(lse); e.part_o = DAF_SEG(part_o); e.part_lse = DAF_SEG(part_lse);
    const float inv_l = l > 0.f ? 1.f / l : 0.f;
    const float lse_val = l > 0.f ? m * DAF_SEG(scale) + logf(l) : -INFINITY;
    // Rows leave through shared memory so that global stores are whole 256-byte runs: each
    // thread parks its own row (16-byte chunks, XOR-swizzled against bank conflicts) in the
    // part of the Q tile that belongs to its warp (Q is dead once the last MMA has completed),
    // then the warp writes its 32 rows out, 16 lanes per row.
    auto park = [&](int chunk, uint4 w) {
        *reinterpret_cast<uint4*>(stage + lane * 256 + ((chunk ^ (lane & 7)) << 4)) = w;
    };
    // copy phase: lanes 0-15 take row rr, lanes 16-31 row rr+1, rr advancing by 2; the row's
    // (token, head) pair is tracked incrementally instead of dividing in the loop
    const int sub = lane >> 4, cidx = lane & 15;
    const int r_first = quad * 32 + sub;
    const int step_t = 2 / e.Gp, step_h = 2 % e.Gp;
    const int n_rows_tile = e.Gp * e.Tt;
    if (a.item_splits == 1 && DAF_SEG(out_tiled)) {
        // Rows in token order: the tile is parked in the layout of a tiled copy (two 64-column halves of
        // 128-byte rows, 16-byte chunks XOR-ed with the row number mod 8 -- the layout the Q tile came in)
        // and leaves by two bulk tensor stores, which clip the rows past the end of the output.
        if (row_valid && e.lse != nullptr) e.lse[(size_t)head * e.n_q + tok] = lse_val;
        const int r = quad * 32 + lane;
        if (has_keys) {
#pragma unroll
            for (int cchunk = 0; cchunk < 4; ++cchunk) {
                uint32_t orr[32];
                tmem_ld32(o_addr + (uint32_t)(cchunk * 32), orr);
                tc_wait_ld();
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint4 w;
                    w.x = pack_bf16(__uint_as_float(orr[v * 8 + 0]) * inv_l, __uint_as_float(orr[v * 8 + 1]) * inv_l);
                    w.y = pack_bf16(__uint_as_float(orr[v * 8 + 2]) * inv_l, __uint_as_float(orr[v * 8 + 3]) * inv_l);
                    w.z = pack_bf16(__uint_as_float(orr[v * 8 + 4]) * inv_l, __uint_as_float(orr[v * 8 + 5]) * inv_l);
                    w.w = pack_bf16(__uint_as_float(orr[v * 8 + 6]) * inv_l, __uint_as_float(orr[v * 8 + 7]) * inv_l);
                    const int c = cchunk * 4 + v;     // 16-byte chunk of the 256-byte row
                    *reinterpret_cast<uint4*>(q_tile + (c >> 3) * kHalfBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = w;
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(rows_parked);
            if (quad == 0) {
                // the first softmax warp waits (bounded) until all four have parked their rows; one lane stores
                bool all = mbar_wait(rows_parked, 0, abort_flag, args.status, 70);
                all = __all_sync(0xFFFFFFFFu, all);
                if (all && lane == 0) {
                    tma_store_3d(tmap_o, q_tile, 0, h0, t0);
                    tma_store_3d(tmap_o, q_tile + kHalfBytes, 64, h0, t0);
                    tma_store_commit();
                    tma_store_wait_read();      // shared memory may be released once the stores have read it
                }
                __syncwarp();
            }
        }
    } else if (a.item_splits == 1) {
        if (row_valid && e.lse != nullptr) e.lse[(size_t)head * e.n_q + tok] = lse_val;
        if (has_keys) {
#pragma unroll
            for (int cchunk = 0; cchunk < 4; ++cchunk) {
                uint32_t orr[32];
                tmem_ld32(o_addr + (uint32_t)(cchunk * 32), orr);
                tc_wait_ld();
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint4 w;
                    w.x = pack_bf16(__uint_as_float(orr[v * 8 + 0]) * inv_l, __uint_as_float(orr[v * 8 + 1]) * inv_l);
                    w.y = pack_bf16(__uint_as_float(orr[v * 8 + 2]) * inv_l, __uint_as_float(orr[v * 8 + 3]) * inv_l);
                    w.z = pack_bf16(__uint_as_float(orr[v * 8 + 4]) * inv_l, __uint_as_float(orr[v * 8 + 5]) * inv_l);
                    w.w = pack_bf16(__uint_as_float(orr[v * 8 + 6]) * inv_l, __uint_as_float(orr[v * 8 + 7]) * inv_l);
                    park(cchunk * 4 + v, w);
                }
            }
            __syncwarp();
            int tok_r = t0 + r_first / e.Gp, head_off = r_first % e.Gp;
#pragma unroll 4
            for (int i = 0; i < 16; ++i) {
                const int rr = 2 * i + sub;
                if (quad * 32 + rr < n_rows_tile && tok_r < e.n_q) {
                    const long long drow = e.dst_rows ? (long long)e.dst_rows[tok_r] : (long long)tok_r;
                    const uint4 w = *reinterpret_cast<const uint4*>(stage + rr * 256 + ((cidx ^ (rr & 7)) << 4));
                    reinterpret_cast<uint4*>(e.out + drow * e.out_row_stride + (long long)(h0 + head_off) * kD)[cidx] = w;
                }
                head_off += step_h; tok_r += step_t;
                if (head_off >= e.Gp) { head_off -= e.Gp; ++tok_r; }
            }
        }
    } else {
        const long long prow0 = a.part_row0 - a.tok_base;
        if (row_valid) e.part_lse[(prow0 + tok) * e.Hq + head] = lse_val;
#pragma unroll
        for (int half = 0; half < 2; ++half) {   // 64 fp32 columns (256 bytes per row) at a time
            if (has_keys) {
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    uint32_t orr[32];
                    tmem_ld32(o_addr + (uint32_t)((half * 2 + cc) * 32), orr);
                    tc_wait_ld();
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        uint4 w;
                        w.x = __float_as_uint(__uint_as_float(orr[v * 4 + 0]) * inv_l);
                        w.y = __float_as_uint(__uint_as_float(orr[v * 4 + 1]) * inv_l);
                        w.z = __float_as_uint(__uint_as_float(orr[v * 4 + 2]) * inv_l);
                        w.w = __float_as_uint(__uint_as_float(orr[v * 4 + 3]) * inv_l);
                        park(cc * 8 + v, w);
                    }
                }
            } else {
#pragma unroll
                for (int v = 0; v < 16; ++v) park(v, make_uint4(0u, 0u, 0u, 0u));
            }
            __syncwarp();
            int tok_r = t0 + r_first / e.Gp, head_off = r_first % e.Gp;
#pragma unroll 4
            for (int i = 0; i < 16; ++i) {
                const int rr = 2 * i + sub;
                if (row_valid_tile && quad * 32 + rr < n_rows_tile && tok_r < e.n_q) {
                    const uint4 w = *reinterpret_cast<const uint4*>(stage + rr * 256 + ((cidx ^ (rr & 7)) << 4));
                    float* prow = e.part_o + ((prow0 + tok_r) * e.Hq + (h0 + head_off)) * kD + half * 64;
                    reinterpret_cast<uint4*>(prow)[cidx] = w;
                }
                head_off += step_h; tok_r += step_t;
                if (head_off >= e.Gp) { head_off -= e.Gp; ++tok_r; }
            }
            __syncwarp();
        }
    }
}

#ifdef DAF_TRACE
extern "C" int daf_dbg_read_trace(void* host, size_t bytes) {
    return (int)cudaMemcpyFromSymbol(host, g_trace, bytes < sizeof(g_trace) ? bytes : sizeof(g_trace));
}
#endif

// ------------------------------------------------------------------------------------------------
// The attention kernel: one 128-row query tile per CTA, two CTAs per SM.
//
// A tile's rows are (token, head) pairs: `Gp` query heads of one KV group times 128/Gp consecutive
// tokens.  Gp = 1 for the packed causal attention; Gp = group size for the question rows, so that
// one pass over the KV cache serves every query head of the group.
//   - one warp issues TMA loads of Q and of K/V sub-tiles of 64 keys into shared-memory rings,
//   - one warp issues tcgen05 MMAs: S = Q K^T into tensor memory, then O += P V with P read back
//     from tensor memory (in both, the warp walks its loop as a whole and an elected lane issues),
//   - four warps run the online softmax, one thread per row, straight out of tensor memory, and
//     write the final rows.
// The keys go through in sub-steps of 64 and S is double-buffered (two 64-column halves of the
// same 128 tensor-memory columns): the logits of sub-step t + 1 are computed while the softmax of
// sub-step t runs, so the softmax warps find their next input ready.  The products O += P_t V_t are
// issued as each P_t arrives, in order; only a row that has to be rescaled waits for the product before
// it to complete (pv_done).  The second CTA of the SM fills what gaps remain.  Final rows in token order
// leave by tiled bulk stores from the dead Q tile.
// Two tiles per CTA sharing every K/V tile (half the shared-memory fill traffic, one CTA per SM)
// measured slower at every size from 1k to 136k tokens and was removed.
constexpr int kSubN = 64;                               // keys per sub-step
constexpr int kSubBytes = kSubN * kD * 2;               // 16 KB: K or V of one sub-step, two 64-column halves
constexpr int kSubHalfBytes = kSubBytes / 2;
constexpr int kAttnThreads = 192;                      // warps 0-3 softmax, warp 4 TMA, warp 5 MMA
constexpr int kGatherWarps = 3;                        // form that fetches K/V rows in place: warps 4, 6 and 7 copy them
constexpr int kAttnThreadsGather = 256;
constexpr int kAttnTmemCols = 256;                     // S (two halves of 64) and O (128)

struct AttnSmem {
    uint64_t q_full;
    uint64_t k_full[2], v_full[2];
    uint64_t s_full[2], p_full[2];
    uint64_t pv_done[2];      // O += P_t V_t has completed: sub-steps alternate between the two barriers
    uint64_t rows_parked;     // epilogue: the four softmax warps have parked their rows for the tiled store
    uint32_t tmem_base;
    int abort_flag;
};
constexpr size_t kAttnSmemBytes = 1024 + 3 * (size_t)kTileBytes + sizeof(AttnSmem);

template <bool kGatherKV>
__global__ void __launch_bounds__(kGatherKV ? kAttnThreadsGather : kAttnThreads, 2)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tmap_q0, const __grid_constant__ CUtensorMap tmap_k0,
                  const __grid_constant__ CUtensorMap tmap_v0, const __grid_constant__ CUtensorMap tmap_q1,
                  const __grid_constant__ CUtensorMap tmap_k1, const __grid_constant__ CUtensorMap tmap_v1,
                  const __grid_constant__ CUtensorMap tmap_o0, const __grid_constant__ CUtensorMap tmap_o1,
                  const AttnArgs args) {
    extern __shared__ unsigned char attn_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(attn_smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char* q_smem = smem;                                 // 32 KB
    unsigned char* k_smem = smem + kTileBytes;                    // two sub-step slots
    unsigned char* v_smem = smem + 2 * (size_t)kTileBytes;        // two sub-step slots
    AttnSmem* sm = reinterpret_cast<AttnSmem*>(smem + 3 * (size_t)kTileBytes);


    if (threadIdx.x == 0) DAF_STAMP(0);
    DAF_KT_BEGIN(0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    CtaWork a;
    decode_work(args, a);
    const int seg_id = a.seg_id;
    const CUtensorMap* tmap_q = seg_id ? &tmap_q1 : &tmap_q0;
    const CUtensorMap* tmap_k = seg_id ? &tmap_k1 : &tmap_k0;
    const CUtensorMap* tmap_v = seg_id ? &tmap_v1 : &tmap_v0;
    DeviceStatus* const status = args.status;
    const int h0 = a.hb * a.Gp;
    const int g_kv = h0 / a.G;
    const int t0 = a.unit * a.Tt;
    const int key_begin = a.j_begin * kBlockN;
    // kGatherKV: the launch has a problem whose K/V rows the producer warp fetches in place through an index (k_src
    // non-null); a form of its own, so that the plain form carries none of that code
    const __nv_bfloat16* const k_src = kGatherKV ? DAF_SEG(k_src) : nullptr;
    const bool kv_gather = kGatherKV && k_src != nullptr;
    const int gather_warp = warp == 4 ? 0 : warp - 5;    // 0, 1, 2 for warps 4, 6, 7 (meaningful only for those)

    // Loads K (kv = 0) or V (kv = 1) of sub-step t into its ring slot (the slot must be free).
    auto issue_kv = [&](int t, int kv) {
        const int slot = t & 1;
        uint64_t* full = kv == 0 ? &sm->k_full[slot] : &sm->v_full[slot];
        unsigned char* dst = (kv == 0 ? k_smem : v_smem) + (size_t)slot * kSubBytes;
        const CUtensorMap* tm = kv == 0 ? tmap_k : tmap_v;
        const int key0 = key_begin + t * kSubN;
        mbar_arrive_expect_tx(full, (uint32_t)kSubBytes);
        tma_load_3d(dst, tm, full, 0, g_kv, key0);
        tma_load_3d(dst + kSubHalfBytes, tm, full, 64, g_kv, key0);
    };
    // The same for K/V rows fetched in place (three warps share the rows of a sub-step, every lane arrives on the
    // slot's barrier): row j of the sub-step is row idx[key0 + j] of
    // the source tensor, copied by cp.async in 16-byte chunks into the layout the tiled load would have produced;
    // rows past the end are zero-filled.  pos_lo / pos_hi: this lane's source rows for sub-tile rows `lane` and
    // `32 + lane` (-1: none).  A copy group is handed to the tensor cores by kv_gather_arrive once it has landed.
    uint64_t* gather_pending = nullptr;          // full-barrier of the copy group committed last
    auto kv_gather_arrive = [&](bool all) {
        if (gather_pending != nullptr) {
            if (all) cp_async_wait_group<0>(); else cp_async_wait_group<1>();
            fence_proxy_async();                 // this lane's landed copies, before the tensor cores read them
            mbar_arrive(gather_pending);
        }
    };
    // Byte offsets (within the K or V tensor) of the 16-byte chunks this lane copies for its warp's pairs of rows of
    // sub-step t: computed once, used for K and for V.  -1: the row lies past the end (zero fill).
    constexpr int kGatherPairs = (32 + kGatherWarps - 1) / kGatherWarps;
    auto gather_offsets = [&](int t, long long (&off)[kGatherPairs]) {
        const int key0 = key_begin + t * kSubN;
        const int rows = DAF_SEG(kv_src_rows);
        const int32_t* kv_idx = DAF_SEG(kv_idx);
        int pos_lo = -1, pos_hi = -1;
        if (key0 + lane < a.n_kv) { const int v = __ldg(kv_idx + key0 + lane); if ((unsigned)v < (unsigned)rows) pos_lo = v; }
        if (key0 + 32 + lane < a.n_kv) { const int v = __ldg(kv_idx + key0 + 32 + lane); if ((unsigned)v < (unsigned)rows) pos_hi = v; }
        const long long row_bytes = (long long)DAF_SEG(kv_heads) * kD * 2;
        const int sub = lane >> 4, ch = lane & 15;
#pragma unroll
        for (int u = 0; u < kGatherPairs; ++u) {
            const int i = gather_warp + u * kGatherWarps;          // pair of rows (2i, 2i + 1)
            const int j = 2 * i + sub;
            const int pos = __shfl_sync(0xFFFFFFFFu, i < 16 ? pos_lo : pos_hi, j & 31);
            off[u] = (i < 32 && pos >= 0) ? (long long)pos * row_bytes + (long long)(g_kv * kD * 2 + ch * 16) : -1;
        }
    };
    auto gather_kv = [&](int t, int kv, const long long (&off)[kGatherPairs]) {
        const int slot = t & 1;
        uint64_t* full = kv == 0 ? &sm->k_full[slot] : &sm->v_full[slot];
        const char* src = reinterpret_cast<const char*>(kv == 0 ? k_src : DAF_SEG(v_src));
        const int sub = lane >> 4, ch = lane & 15;
        // this lane's chunk of row j lands at half (ch >> 3), row j, chunk ((ch & 7) ^ (j & 7)); j & 7 = ((2 i) & 7) | sub
        const uint32_t dst = smem_u32((kv == 0 ? k_smem : v_smem) + (size_t)slot * kSubBytes) +
                             (uint32_t)((ch >> 3) * kSubHalfBytes + sub * 128);
        const uint32_t x = (uint32_t)((ch & 7) ^ sub);
#pragma unroll
        for (int u = 0; u < kGatherPairs; ++u) {
            const int i = gather_warp + u * kGatherWarps;
            if (i < 32)
                cp_async16(dst + (uint32_t)(i * 256) + ((x ^ (uint32_t)((2 * i) & 7)) << 4),
                           src + (off[u] < 0 ? 0 : off[u]), off[u] < 0 ? 0u : 16u);
        }
        cp_async_commit();
        kv_gather_arrive(false);                 // the group before this one has landed (or is waited for here)
        gather_pending = full;
    };
    // Set-up.  The producer thread prepares the barriers and at once starts the loads that need no free
    // slot (Q and the first two sub-steps), so that their latency overlaps the rest of the set-up: the
    // status check (a global read) and the tensor-memory allocation.
    // Everything up to the wait below touches no memory an earlier kernel writes, so with programmatic
    // dependent launch it runs while the kernel launched just before (gather / hybrid-cache update) drains.
    __shared__ int skip_cta;
    const int32_t* const q_idx = DAF_SEG(q_idx);     // non-null: the softmax warps fetch the Q rows themselves
    if (warp == 5) {
        tmem_alloc(&sm->tmem_base, kAttnTmemCols);
        tmem_relinquish();
    }
    if (warp == 4 && lane == 0) {
        mbar_init(&sm->q_full, q_idx != nullptr ? 4 : 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&sm->k_full[s], kv_gather ? 32 * kGatherWarps : 1); mbar_init(&sm->v_full[s], kv_gather ? 32 * kGatherWarps : 1);
            mbar_init(&sm->s_full[s], 1); mbar_init(&sm->p_full[s], 4);
        }
        mbar_init(&sm->pv_done[0], 1); mbar_init(&sm->pv_done[1], 1);
        mbar_init(&sm->rows_parked, 4);
        sm->abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(tmap_k);
        tma_prefetch_desc(tmap_v);
        if (q_idx == nullptr) tma_prefetch_desc(tmap_q);
    }
    pdl_wait();                // from here on: inputs that the kernel launched just before may have written
    // sub-steps of this item: the keys of its range that the tile's last token may see
    int n_t = 0;
    if (a.unit < a.n_tb) {
        const int max_tok = min(a.n_q, t0 + a.Tt) - 1;
        const long long last_key = a.q_pos ? (long long)__ldg(a.q_pos + max_tok) : (long long)max_tok + a.causal_off;
        long long hi = min((long long)a.n_kv, last_key + 1);
        hi = min(hi, (long long)a.j_end * kBlockN);
        if (hi > key_begin) n_t = (int)((hi - key_begin + kSubN - 1) / kSubN);
    }
    if (warp == 4 && lane == 0) {
        if (n_t > 0) {
            if (q_idx == nullptr) {
                mbar_arrive_expect_tx(&sm->q_full, 2u * 128u * (uint32_t)(a.Gp * a.Tt));
                tma_load_3d(q_smem, tmap_q, &sm->q_full, 0, h0, t0);
                tma_load_3d(q_smem + kHalfBytes, tmap_q, &sm->q_full, 64, h0, t0);
            }
            if (!kv_gather)
                for (int t = 0; t < 2 && t < n_t; ++t) { issue_kv(t, 0); issue_kv(t, 1); }
        }
    }
    if (q_idx != nullptr && n_t > 0 && warp < 4) {
        const int quad = warp;
        // Q rows of the condensed sequence straight from the unpacked tensor: each warp fetches its 32
        // rows (16 lanes per 256-byte row) into the layout the TMA load would have produced
        // (two 64-column halves of 128-byte rows, 16-byte chunks XOR-ed with the row number mod 8).
        const __nv_bfloat16* q_src = DAF_SEG(q_src);
        const int q_src_rows = DAF_SEG(q_src_rows), Hq = DAF_SEG(Hq);
        const int sub = lane >> 4, cidx = lane & 15;
        uint4 w[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int tokr = t0 + quad * 32 + 2 * i + sub;
            w[i] = make_uint4(0u, 0u, 0u, 0u);
            if (tokr < a.n_q) {
                const int src = __ldg(q_idx + tokr);
                if ((unsigned)src < (unsigned)q_src_rows)   // a bad position is reported by the gather kernel
                    w[i] = __ldg(reinterpret_cast<const uint4*>(q_src + ((size_t)src * Hq + h0) * kD) + cidx);
            }
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int rr = quad * 32 + 2 * i + sub;
            *reinterpret_cast<uint4*>(q_smem + (cidx >> 3) * kHalfBytes + rr * 128 + (((cidx & 7) ^ (rr & 7)) << 4)) = w[i];
        }
        fence_proxy_async();
    }
    // a CTA of this grid (or an earlier kernel sharing the workspace) has already given up: do nothing
    if (threadIdx.x == 0) skip_cta = (status != nullptr && *reinterpret_cast<volatile int*>(&status->code) != 0) ? 1 : 0;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm->tmem_base;
    volatile int* abort_flag = &sm->abort_flag;
    const bool skip = skip_cta != 0;
    if (threadIdx.x == 0) DAF_STAMP(1);

    if (skip) {
        // nothing is computed; the loads already under way get a bounded chance to land before the CTA retires
        if (warp == 4 && lane == 0 && n_t > 0 && !kv_gather) {
            for (int i = 0; i < 4096 && !mbar_try_wait(&sm->q_full, 0); ++i) {}
            for (int s = 0; s < 2 && s < n_t; ++s) {
                for (int i = 0; i < 4096 && !mbar_try_wait(&sm->k_full[s], 0); ++i) {}
                for (int i = 0; i < 4096 && !mbar_try_wait(&sm->v_full[s], 0); ++i) {}
            }
        }
    } else if (kv_gather && (warp == 4 || warp >= 6)) {
        // ------------------------------------------------------------ producers of the form that fetches K/V rows in place
        // (all sub-steps, after the set-up barrier: the barriers must be ready before three warps arrive on them)
        bool ok = true;
        for (int t = 0; t < n_t && ok; ++t) {
            const int slot = t & 1;
            const uint32_t round = (uint32_t)(t >> 1);
            long long off[kGatherPairs];
            gather_offsets(t, off);
            for (int kv = 0; kv < 2 && ok; ++kv) {
                if (t >= 2) {
                    uint64_t* empty = kv == 0 ? &sm->s_full[slot] : &sm->pv_done[slot];
                    ok = mbar_wait(empty, (round - 1) & 1u, abort_flag, status, 14 + 2 * kv + slot);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                }
                if (ok) gather_kv(t, kv, off);
                __syncwarp();
            }
        }
        kv_gather_arrive(true);   // the last copy group (also on the way out after a give-up: copies always land)
    } else if (warp == 4) {
        // ------------------------------------------------------------ TMA producer (the rest of the sub-steps)
        if (n_t > 2) {   // the whole warp walks the loop, one elected lane issues (uniform control flow)
            bool ok = true;
            for (int t = 2; t < n_t && ok; ++t) {
                const int slot = t & 1;
                const uint32_t round = (uint32_t)(t >> 1);
                for (int kv = 0; kv < 2 && ok; ++kv) {
                    // a K slot is free once the logits read from it are complete, a V slot once its product is:
                    // the barriers the softmax warps wait on say exactly that, so the issuer commits nothing extra
                    uint64_t* empty = kv == 0 ? &sm->s_full[slot] : &sm->pv_done[slot];
                    ok = mbar_wait(empty, (round - 1) & 1u, abort_flag, status, 10 + 2 * kv + slot);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (ok && elect_one()) issue_kv(t, kv);
                    __syncwarp();
                }
            }
            if (!ok && lane == 0) {
                // give loads already in flight a bounded chance to land before the CTA retires
                for (int s = 0; s < 2; ++s) {
                    for (int i = 0; i < 4096 && !mbar_try_wait(&sm->k_full[s], 0) && !mbar_try_wait(&sm->k_full[s], 1); ++i) {}
                    for (int i = 0; i < 4096 && !mbar_try_wait(&sm->v_full[s], 0) && !mbar_try_wait(&sm->v_full[s], 1); ++i) {}
                }
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ MMA issuer
        // The whole warp walks the loop and waits on the barriers, one elected lane issues: control flow
        // stays uniform across the warp, so the operand descriptors can live in uniform registers.
        if (n_t > 0) {
            constexpr uint32_t idesc_qk = make_idesc_bf16(kBlockM, kSubN, 0);
            constexpr uint32_t idesc_pv = make_idesc_bf16(kBlockM, kD, 1);
            const uint32_t qa = smem_u32(q_smem);
            // S_b = Q K_t^T for the 64 keys in K slot b (= t & 1)
            // every operand descriptor is fixed for the whole item: they are built once, ahead of the loop
            uint64_t qd[kD / 16], kd[2][kD / 16], vd[2][kSubN / 16];
#pragma unroll
            for (int kk = 0; kk < kD / 16; ++kk) {
                qd[kk] = make_smem_desc(qa + (uint32_t)((kk & 3) * 32 + (kk >> 2) * kHalfBytes), 16, 1024);
#pragma unroll
                for (int b = 0; b < 2; ++b)
                    kd[b][kk] = make_smem_desc(smem_u32(k_smem + (size_t)b * kSubBytes) + (uint32_t)((kk & 3) * 32 + (kk >> 2) * kSubHalfBytes), 16, 1024);
            }
#pragma unroll
            for (int kk = 0; kk < kSubN / 16; ++kk)
#pragma unroll
                for (int b = 0; b < 2; ++b)
                    vd[b][kk] = make_smem_desc(smem_u32(v_smem + (size_t)b * kSubBytes) + (uint32_t)kk * 2048u, kSubHalfBytes, 1024);
            auto issue_qk = [&](int b) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)
                    tc_mma_ss(tmem + (uint32_t)(b * kSubN), qd[kk], b ? kd[1][kk] : kd[0][kk], idesc_qk, kk > 0 ? 1u : 0u);
            };
            // O (+)= P_b V_t for the 64 keys in V slot b; P (bf16) sits in the first 32 columns of S_b
            auto issue_pv = [&](int b, bool first) {
#pragma unroll
                for (int kk = 0; kk < kSubN / 16; ++kk)
                    tc_mma_ts(tmem + (uint32_t)kBlockN, tmem + (uint32_t)(b * kSubN + kk * 8), b ? vd[1][kk] : vd[0][kk], idesc_pv,
                              (first && kk == 0) ? 0u : 1u);
            };
            bool ok = mbar_wait(&sm->q_full, 0, abort_flag, status, 20);
            ok = __all_sync(0xFFFFFFFFu, ok);
            for (int t = 0; t < 2 && t < n_t && ok; ++t) {   // the first two S tiles
                ok = mbar_wait(&sm->k_full[t], 0, abort_flag, status, 30 + t);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
                    issue_qk(t);
                    tc_commit(&sm->s_full[t]);
                }
                __syncwarp();
            }
            for (int t = 0; t < n_t && ok; ++t) {
                const int b = t & 1;
                const uint32_t par = (uint32_t)((t >> 1) & 1);
                ok = mbar_wait(&sm->v_full[b], par, abort_flag, status, 32 + b);
                if (ok) ok = mbar_wait(&sm->p_full[b], par, abort_flag, status, 40 + b);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
                    issue_pv(b, t == 0);
                    tc_commit(&sm->pv_done[b]);
                }
                __syncwarp();
                if (t + 2 < n_t) {
                    ok = mbar_wait(&sm->k_full[b], (uint32_t)(((t + 2) >> 1) & 1), abort_flag, status, 34 + b);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    if (elect_one()) {
                        issue_qk(b);
                        tc_commit(&sm->s_full[b]);
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------ softmax + epilogue, one row per thread
        const int quad = warp;
        const int r = quad * 32 + lane;
        const int tok = t0 + r / a.Gp;
        const int head = h0 + r % a.Gp;
        const bool row_valid_tile = (n_t > 0 || a.item_splits > 1) && (a.unit < a.n_tb);
        const bool row_valid = (r < a.Gp * a.Tt) && (tok < a.n_q) && row_valid_tile;
        const long long lim_ll = (a.q_pos && tok < a.n_q) ? (long long)__ldg(a.q_pos + tok) : (long long)tok + a.causal_off;
        const int limit = row_valid ? (int)min(lim_ll, (long long)a.n_kv - 1) : -1;   // last visible key
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const uint32_t s_addr = tmem + lane_addr;
        const uint32_t o_addr = tmem + lane_addr + (uint32_t)kBlockN;
        const float c = a.scale_log2;

        if (q_idx != nullptr && n_t > 0 && lane == 0) mbar_arrive(&sm->q_full);   // this warp's Q rows were stored before the set-up barrier
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        DAF_LAP_DECL;
        for (int t = 0; t < n_t; ++t) {
            const int b = t & 1;
            ok = mbar_wait(&sm->s_full[b], (uint32_t)((t >> 1) & 1), abort_flag, status, 50 + b);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            if (threadIdx.x == 0 && t == 0) DAF_STAMP(2);
            DAF_LAP(lap_s);
            const float alpha = softmax_core<2>(s_addr + (uint32_t)(b * kSubN), key_begin + t * kSubN, limit, c, m, l);
            DAF_LAP(lap_soft);
            if (t > 0 && __any_sync(0xFFFFFFFFu, alpha != 1.f)) {
                // A row of this warp has to be rescaled: O may be touched only once the product before has
                // completed.  (Rare: the running maximum is kept stale up to 2^8.  When no row needs it the warp
                // does not wait at all -- the products run in issue order, so P_t may be handed over while
                // O += P_{t-1} V_{t-1} is still under way.)  Sub-steps alternate between two barriers, so the
                // phase waited for is unambiguous although the warp has not observed every phase.
                ok = mbar_wait(&sm->pv_done[(t - 1) & 1], (uint32_t)(((t - 1) >> 1) & 1), abort_flag, status, 60);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                rescale_o(o_addr, alpha);
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm->p_full[b]);   // one arrival per warp: all its rows of P (and of O) are in place
            DAF_LAP(lap_pv);
        }
        if (threadIdx.x == 0) DAF_STAMP(3);
        // ---- epilogue
        if (ok && n_t > 0) {
            ok = mbar_wait(&sm->pv_done[(n_t - 1) & 1], (uint32_t)(((n_t - 1) >> 1) & 1), abort_flag, status, 61);
            ok = __all_sync(0xFFFFFFFFu, ok);
        }
        if (ok) {
            tc_fence_after();
            write_rows(args, a, t0, n_t > 0, row_valid, row_valid_tile, tok, head, h0, q_smem, seg_id ? &tmap_o1 : &tmap_o0,
                       &sm->rows_parked, abort_flag, o_addr, quad, lane, m, l);
        }
#ifdef DAF_TRACE
        if (threadIdx.x == 0) {
            const unsigned cta = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
            if (cta < 65536u) {
                long long* t = g_laps + 8 * cta;
                const long long now = clock64();
                t[0] = now - lap_begin; t[1] = lap_s; t[2] = lap_soft; t[3] = lap_pv; t[4] = now - lap_t; t[5] = n_t;
            }
        }
#endif
    }

    if (threadIdx.x == 0) DAF_STAMP(4);
    // Only now may the dependent kernel (the merge of the key ranges) start launching: its CTAs wait for this
    // whole grid, and while they wait they hold registers and thread slots that CTAs of this grid could use.
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem, kAttnTmemCols);
    }
    DAF_KT_END(0);
#ifdef DAF_TRACE
    if (threadIdx.x == 0) {
        DAF_STAMP(5);
        const unsigned cta = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
        if (cta < 65536u) {
            g_trace[8 * cta + 6] = (unsigned long long)n_t;
            unsigned smid; asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
            g_trace[8 * cta + 7] = ((unsigned long long)smid << 32) | (unsigned long long)sm->tmem_base;
        }
    }
#endif
}


#undef DAF_SEG

// Merge of partial results: one warp per (token, head) row.  A launch merges the rows of up to two
// problems (those of s0 first).  A row's partials sit `stride` rows apart; how many there are is the
// same for every row (n_splits) or, for a problem cut into balanced ranges, follows from its unit.
struct CombineSeg {
    const float* part_o; const float* part_lse;
    int n_q, Hq;
    int tok_first;       // rows of tokens below this were written in final form by the attention kernel
    int n_rows;          // (n_q - tok_first) * Hq
    int n_splits;        // > 0: every row has this many partials, n_q * Hq rows apart
    int unit_tokens, chunk;   // n_splits == 0: tokens per unit, units per group (see SegArgs)
    __nv_bfloat16* out; long long out_row_stride; const int32_t* dst_rows; float* lse;
};

__global__ void __launch_bounds__(256)
attn_combine_kernel(const CombineSeg s0, const CombineSeg s1) {
    DAF_KT_BEGIN(2);
    pdl_wait();                // partial results come from the attention kernel launched just before
    DAF_KT_BEGIN(3);
    int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const bool second = row >= s0.n_rows;
    if (second) row -= s0.n_rows;
#define DAF_CS(field) (second ? s1.field : s0.field)
    if (row >= DAF_CS(n_rows)) return;
    const int Hq = DAF_CS(Hq), n_q = DAF_CS(n_q);
    const int tok = DAF_CS(tok_first) + row / Hq, head = row % Hq;
    int n_splits = DAF_CS(n_splits);
    size_t first, stride;      // in rows of the partial arrays
    if (n_splits > 0) {
        first = (size_t)tok * Hq + head;
        stride = (size_t)n_q * Hq;
    } else {
        const int ut = DAF_CS(unit_tokens), chunk = DAF_CS(chunk);
        const int unit = tok / ut, g = unit / chunk;
        n_splits = g + 1;
        const int slot0 = chunk * g * (g + 1) / 2 + (unit - g * chunk) * (g + 1);
        first = ((size_t)slot0 * ut + (size_t)(tok - unit * ut)) * Hq + head;
        stride = (size_t)ut * Hq;
    }
    const float* part_o = DAF_CS(part_o);
    const float* part_lse = DAF_CS(part_lse);
    // lane s holds the log-sum-exp of partial s (at most 32 of them), so all of them are fetched at once;
    // the first eight partial rows are requested in the same breath, before the weights are known
    const float4* src = reinterpret_cast<const float4*>(part_o + first * kD) + lane;
    const float my_lse = lane < n_splits ? part_lse[first + (size_t)lane * stride] : -INFINITY;
    float4 head_v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
        head_v[u] = u < n_splits ? __ldcs(src + (size_t)u * stride * (kD / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
    float mx = my_lse;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    const float my_w = (my_lse == -INFINITY) ? 0.f : __expf(my_lse - mx);
    float wsum = my_w;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wsum += __shfl_xor_sync(0xFFFFFFFFu, wsum, o);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const float w = __shfl_sync(0xFFFFFFFFu, my_w, u);     // zero for u >= n_splits
        acc.x += w * head_v[u].x; acc.y += w * head_v[u].y; acc.z += w * head_v[u].z; acc.w += w * head_v[u].w;
    }
    int s = 8;
    for (; s + 4 <= n_splits; s += 4) {
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = __ldcs(src + (size_t)(s + u) * stride * (kD / 4));
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float w = __shfl_sync(0xFFFFFFFFu, my_w, s + u);
            acc.x += w * v[u].x; acc.y += w * v[u].y; acc.z += w * v[u].z; acc.w += w * v[u].w;
        }
    }
    for (; s < n_splits; ++s) {
        const float4 v = __ldcs(src + (size_t)s * stride * (kD / 4));
        const float w = __shfl_sync(0xFFFFFFFFu, my_w, s);
        acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
    }
    const float inv = wsum > 0.f ? 1.f / wsum : 0.f;
    const int32_t* dst_rows = DAF_CS(dst_rows);
    const long long drow = dst_rows ? (long long)dst_rows[tok] : (long long)tok;
    uint2 w2;
    w2.x = pack_bf16(acc.x * inv, acc.y * inv);
    w2.y = pack_bf16(acc.z * inv, acc.w * inv);
    reinterpret_cast<uint2*>(DAF_CS(out) + drow * DAF_CS(out_row_stride) + (long long)head * kD)[lane] = w2;
    float* lse = DAF_CS(lse);
    if (lse != nullptr && lane == 0) lse[(size_t)head * n_q + tok] = wsum > 0.f ? mx + logf(wsum) : -INFINITY;
    DAF_KT_END(2);
#undef DAF_CS
}

// ----------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || p == nullptr) {
            set_cuda_error(e != cudaSuccess ? e : cudaErrorUnknown);
            return nullptr;
        }
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [tokens, heads, 128] bf16 viewed as (d, head, token); a box is 64 columns x box_heads x box_tokens,
// written to shared memory as 128-byte rows with the 128-byte swizzle.  row_stride_bytes = 0: rows are contiguous.
// Encoding a map costs about a microsecond of host time and a layer needs eight, so each host thread keeps
// the maps it encoded last, keyed by everything that goes into them (no lock, nothing shared).
namespace {
struct TmapKey {
    const void* base; int tokens, heads, box_heads, box_tokens; long long row_stride;
    bool operator==(const TmapKey& o) const {
        return base == o.base && tokens == o.tokens && heads == o.heads && box_heads == o.box_heads &&
               box_tokens == o.box_tokens && row_stride == o.row_stride;
    }
};
struct TmapSlot { TmapKey key; CUtensorMap map; bool used; };
constexpr int kTmapCacheSlots = 1024;      // direct-mapped; a colliding entry is simply re-encoded
}  // namespace

static int make_tmap(CUtensorMap* m, const void* base, int tokens, int heads, int box_heads, int box_tokens,
                     long long row_stride_bytes = 0) {
    static thread_local std::vector<TmapSlot> cache;
    if (cache.empty()) cache.resize(kTmapCacheSlots, TmapSlot{{nullptr, 0, 0, 0, 0, 0}, {}, false});
    const TmapKey key{base, tokens, heads, box_heads, box_tokens, row_stride_bytes};
    size_t h = reinterpret_cast<uintptr_t>(base) >> 8;
    h = h * 1000003u + (size_t)tokens * 31u + (size_t)box_tokens * 7u + (size_t)box_heads;
    TmapSlot& slot = cache[h % kTmapCacheSlots];
    if (slot.used && slot.key == key) { *m = slot.map; return DAF_OK; }
    EncodeTiledFn fn = get_encode_fn();
    if (fn == nullptr) return DAF_ERR_CUDA;
    cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)heads, (cuuint64_t)tokens};
    cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)(row_stride_bytes > 0 ? row_stride_bytes : (long long)heads * kD * 2)};
    cuuint32_t box[3] = {64u, (cuuint32_t)box_heads, (cuuint32_t)box_tokens};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_cuda_error(cudaErrorInvalidValue); return DAF_ERR_CUDA; }
    slot.key = key; slot.map = *m; slot.used = true;
    return DAF_OK;
}

static int set_kernel_attributes() {
    // per device, set once; concurrent first calls may both set it (the same value), which is harmless
    static std::atomic<bool> attr_done[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_done[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(attn_fwd_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttnSmemBytes);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attn_fwd_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttnSmemBytes);
        if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
        attr_done[dev].store(true, std::memory_order_release);
    }
    return DAF_OK;
}

// SMs of the current device (asked once per device; 148 on B200).  Planning runs on the host and also
// without a device (workspace sizing in CPU-only processes): then the B200 figure is used.
static int num_sms() {
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return kNumSMsDefault; }
    int n = cached[dev].load(std::memory_order_acquire);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            n = kNumSMsDefault;
        }
        cached[dev].store(n, std::memory_order_release);
    }
    return n;
}

// How a single problem is cut into CTAs: one per (head block, token block), and for the question rows,
// where there are few query tiles and a long KV axis, also per range of the KV axis.

AttnPlan plan_attention(int n_q, int n_kv, int Hq, int G, int causal_off, bool pack_group, bool allow_split) {
    AttnPlan pl;
    pl.Gp = pack_group ? G : 1;
    if (pl.Gp > 128) pl.Gp = 1;
    pl.Tt = kBlockM / pl.Gp;
    pl.n_tb = (n_q + pl.Tt - 1) / pl.Tt;
    pl.head_blocks = Hq / pl.Gp;
    long long kv_hi = (long long)n_q - 1 + causal_off + 1;
    if (kv_hi > n_kv) kv_hi = n_kv;
    const int total_tiles = kv_hi > 0 ? (int)((kv_hi + kBlockN - 1) / kBlockN) : 0;
    pl.n_splits = 1;
    pl.tiles_per_split = total_tiles > 0 ? total_tiles : 1;
    if (allow_split && total_tiles > 1) {
        const int ctas = pl.n_tb * pl.head_blocks;
        const int slots = num_sms() * 2;
        int want = ctas > 0 ? slots / ctas : 1;
        if (want > kMaxSplits) want = kMaxSplits;
        if (want > total_tiles) want = total_tiles;
        if (want > 1) {
            pl.tiles_per_split = (total_tiles + want - 1) / want;
            pl.n_splits = (total_tiles + pl.tiles_per_split - 1) / pl.tiles_per_split;
        }
    }
    return pl;
}

size_t attn_partial_bytes(int n_q, int Hq, int n_splits) {
    if (n_splits <= 1) return 0;
    size_t o = (size_t)n_splits * n_q * Hq * kD * sizeof(float);
    size_t l = ((size_t)n_splits * n_q * Hq * sizeof(float) + 255) / 256 * 256;
    return o + l;
}

// Number of (unit, range) slots of units [0, n_units) when groups of `chunk` units are cut into 1, 2, 3, ... ranges.
static int slots_before(int n_units, int chunk) {
    const int g = n_units / chunk;
    return chunk * g * (g + 1) / 2 + (n_units - g * chunk) * (g + 1);
}

// Steps 2 and 3 of one layer as one list of work items.  Two things are free: into how many balanced
// ranges the long causal chains of the important-token stage are cut (`chunk`), and into how many KV
// ranges the question rows are cut.  Finer ranges balance the 296 CTA slots better but cost a fixed
// time per item, partial-result traffic and a longer merge, and the optimum jumps around with the tile
// counts.  So the choice is made by replaying the hardware's dispatch (items in grid order onto the
// slot that frees first) for a handful of candidates with a three-constant cost model and keeping the
// cheapest; the result is cached per problem shape.
namespace {
constexpr float kCostItemUs = 7.0f;        // set-up, first logits and row epilogue of an item (5-6 us alone; fitted)
constexpr float kCostSubStepUs = 1.05f;    // 64 keys through one tile with two CTAs per SM (measured 0.95-1.1 us)
constexpr float kCostMergeUs = 2.0f;       // merge launch
constexpr float kCostMergeUsPerMB = 0.15f; // plus re-reading the partial rows of the question ranges (fitted together with the item cost)
constexpr float kCostMergeUsPerMBCut = 0.45f;  // partial rows of cut causal chains (measured: 7.0 us for 14.8 MB, 13.3 for 25, 42.6 for 96)

int g_force_chunk = 0, g_force_splits_q = 0;   // tuning builds can pin the choice
float g_last_predicted_us = 0.f;

struct JointShape { int k, L_q, L_d, Hq, G; };
bool operator<(const JointShape& a, const JointShape& b) {
    if (a.k != b.k) return a.k < b.k;
    if (a.L_q != b.L_q) return a.L_q < b.L_q;
    if (a.L_d != b.L_d) return a.L_d < b.L_d;
    if (a.Hq != b.Hq) return a.Hq < b.Hq;
    return a.G < b.G;
}

// Fills the fields of `jp` that follow from (chunk, n_splits_q).
void set_choice(JointPlan& jp, int chunk, int n_splits_q, int L_q, int L_d, int Hq) {
    if (chunk < (jp.n_tb_i + 31) / 32) chunk = (jp.n_tb_i + 31) / 32;   // at most 32 ranges per token block
    if (chunk < 1) chunk = 1;
    if (chunk > jp.n_tb_i) chunk = jp.n_tb_i;
    jp.chunk = chunk;
    jp.n_slots = slots_before(jp.n_tb_i, chunk);
    jp.part_bytes_i = 0;
    if (chunk < jp.n_tb_i) {
        const size_t rows = (size_t)jp.n_slots * kBlockM * Hq;
        jp.part_bytes_i = rows * kD * sizeof(float) + (rows * sizeof(float) + 255) / 256 * 256;
    }
    jp.items_i = Hq * jp.n_slots;
    const int tiles_q = (L_d + L_q + kBlockN - 1) / kBlockN;
    if (n_splits_q < 1) n_splits_q = 1;
    jp.tiles_per_split_q = (tiles_q + n_splits_q - 1) / n_splits_q;
    jp.n_splits_q = (tiles_q + jp.tiles_per_split_q - 1) / jp.tiles_per_split_q;
    jp.items_q = jp.head_blocks_q * jp.n_tb_q * jp.n_splits_q;
    jp.part_bytes_q = attn_partial_bytes(L_q, Hq, jp.n_splits_q);
}

// Predicted time of the attention launch + merge for a filled plan, in microseconds.
float predict_us(const JointPlan& jp, int k, int L_q, int L_d, int Hq) {
    const int slots = num_sms() * 2;
    std::priority_queue<float, std::vector<float>, std::greater<float>> free_at;
    for (int i = 0; i < slots; ++i) free_at.push(0.f);
    float makespan = 0.f;
    auto run = [&](int count, int tiles) {
        const float cost = kCostItemUs + kCostSubStepUs * 2.f * (float)tiles;
        for (int i = 0; i < count; ++i) {
            const float t = free_at.top() + cost;
            free_at.pop();
            free_at.push(t);
            if (t > makespan) makespan = t;
        }
    };
    // question items: split-major, token blocks from the last one down, head blocks together
    for (int s = 0; s < jp.n_splits_q; ++s)
        for (int u = jp.n_tb_q - 1; u >= 0; --u) {
            const int last_tok = (u + 1) * jp.Tt_q < L_q ? (u + 1) * jp.Tt_q : L_q;
            const int tiles_total = (L_d + last_tok + kBlockN - 1) / kBlockN;
            int tiles = tiles_total - s * jp.tiles_per_split_q;
            if (tiles > jp.tiles_per_split_q) tiles = jp.tiles_per_split_q;
            if (tiles > 0) run(jp.head_blocks_q, tiles);
        }
    // important-token items: slots from the top down, all heads together
    size_t part_rows_i = 0;
    for (int slot = jp.n_slots - 1; slot >= 0; --slot) {
        int g = 0;
        while (jp.chunk * (g + 1) * (g + 2) / 2 <= slot) ++g;
        const int rem = slot - jp.chunk * g * (g + 1) / 2;
        const int unit = g * jp.chunk + rem / (g + 1), range = rem % (g + 1);
        const int n_tiles = unit + 1 < jp.n_tb_i ? unit + 1 : jp.n_tb_i;
        run(Hq, (range + 1) * n_tiles / (g + 1) - range * n_tiles / (g + 1));
        if (g >= 1) part_rows_i += (size_t)kBlockM * Hq;
    }
    (void)k;
    const float merge_us = kCostMergeUs + kCostMergeUsPerMB * (float)jp.part_bytes_q / 1e6f +
                           kCostMergeUsPerMBCut * (float)(part_rows_i * 516) / 1e6f;
    const bool merges = jp.n_splits_q > 1 || jp.chunk < jp.n_tb_i;
    return makespan + (merges ? merge_us : 0.f);
}
}  // namespace

JointPlan plan_joint(int k, int L_q, int L_d, int Hq, int G) {
    static std::mutex mu;
    static std::map<JointShape, JointPlan> cache;
    const JointShape shape{k, L_q, L_d, Hq, G};
    const bool forced = g_force_chunk > 0 || g_force_splits_q > 0;
    // a layer loop asks for the same shape over and over: each thread keeps its last answer (no lock)
    static thread_local bool have_last = false;
    static thread_local JointShape last_shape;
    static thread_local JointPlan last_plan;
    if (!forced && have_last && !(shape < last_shape) && !(last_shape < shape)) return last_plan;
    if (!forced) {
        std::lock_guard<std::mutex> lock(mu);
        auto it = cache.find(shape);
        if (it != cache.end()) { last_shape = shape; last_plan = it->second; have_last = true; return it->second; }
    }
    JointPlan jp;
    jp.n_tb_i = (k + kBlockM - 1) / kBlockM;
    jp.Gp_q = G > 128 ? 1 : G;
    jp.Tt_q = kBlockM / jp.Gp_q;
    jp.n_tb_q = (L_q + jp.Tt_q - 1) / jp.Tt_q;
    jp.head_blocks_q = Hq / jp.Gp_q;
    const int tiles_q = (L_d + L_q + kBlockN - 1) / kBlockN;
    if (forced) {
        set_choice(jp, g_force_chunk > 0 ? g_force_chunk : jp.n_tb_i, g_force_splits_q > 0 ? g_force_splits_q : 1, L_q, L_d, Hq);
        g_last_predicted_us = predict_us(jp, k, L_q, L_d, Hq);
        return jp;
    }
    // candidates: the causal chains whole, or cut so that the longest has 2..6 ranges; every distinct
    // number of question ranges up to 32
    JointPlan best = jp;
    float best_us = -1.f;
    for (int m = 1; m <= 6; ++m) {
        const int chunk = (jp.n_tb_i + m - 1) / m;
        if (m > 1 && chunk == (jp.n_tb_i + m - 2) / (m - 1)) continue;   // same cut as the previous candidate
        int last_tps = -1;
        for (int n = 1; n <= kMaxSplits && n <= tiles_q; ++n) {
            JointPlan cand = jp;
            set_choice(cand, chunk, n, L_q, L_d, Hq);
            if (cand.tiles_per_split_q == last_tps) continue;
            last_tps = cand.tiles_per_split_q;
            if (cand.part_bytes_i > ((size_t)256 << 20)) continue;   // partials of a large problem: not worth their memory
            const float us = predict_us(cand, k, L_q, L_d, Hq);
            if (best_us < 0.f || us < best_us) { best_us = us; best = cand; }
        }
    }
    g_last_predicted_us = best_us;
    std::lock_guard<std::mutex> lock(mu);
    cache[shape] = best;
    last_shape = shape; last_plan = best; have_last = true;
    return best;
}

#if defined(DAF_TRACE) || defined(DAF_TUNE)     // tuning builds: pin the planner's choice, read its prediction
extern "C" void daf_dbg_joint_force(int chunk, int n_splits_q) { g_force_chunk = chunk; g_force_splits_q = n_splits_q; }
extern "C" float daf_dbg_joint_predicted_us(void) { return g_last_predicted_us; }
extern "C" void daf_dbg_joint_plan(int k, int L_q, int L_d, int Hq, int G, int* out) {
    const JointPlan jp = plan_joint(k, L_q, L_d, Hq, G);
    out[0] = jp.chunk; out[1] = jp.n_tb_i; out[2] = jp.n_splits_q; out[3] = jp.items_i + jp.items_q;
}
#endif

static void fill_problem(SegArgs* s, int n_q, int n_kv, int Hq, int G, int Gp, int causal_off, const int32_t* q_pos,
                         float scale, void* out, long long out_row_stride_bytes, const int32_t* dst_rows, float* lse) {
    s->n_q = n_q; s->n_kv = n_kv; s->Hq = Hq; s->G = G;
    s->Gp = Gp; s->Tt = kBlockM / Gp; s->n_tb = (n_q + s->Tt - 1) / s->Tt;
    s->causal_off = causal_off;
    s->q_pos = q_pos;
    s->head_blocks = Hq / Gp;
    s->scale = scale; s->scale_log2 = scale * 1.4426950408889634f;
    s->out = reinterpret_cast<__nv_bfloat16*>(out);
    s->out_row_stride = out_row_stride_bytes / 2;
    s->dst_rows = dst_rows;
    s->lse = lse;
}

static void fill_combine(CombineSeg* c, const SegArgs& s) {
    const int unit_tokens = kBlockM;   // packed causal attention has one head per tile: a unit is 128 tokens
    c->part_o = s.part_o; c->part_lse = s.part_lse;
    c->n_q = s.n_q; c->Hq = s.Hq;
    c->n_splits = s.chunk == 0 ? s.n_splits : 0;
    c->unit_tokens = unit_tokens; c->chunk = s.chunk > 0 ? s.chunk : 1;
    c->tok_first = 0;
    if (s.chunk == 0 && s.n_splits <= 1) c->tok_first = s.n_q;                    // nothing to merge
    if (s.chunk > 0) c->tok_first = s.chunk * unit_tokens < s.n_q ? s.chunk * unit_tokens : s.n_q;
    c->n_rows = (s.n_q - c->tok_first) * s.Hq;
    c->out = s.out; c->out_row_stride = s.out_row_stride; c->dst_rows = s.dst_rows; c->lse = s.lse;
}

static int launch_combine(const CombineSeg& c0, const CombineSeg& c1, cudaStream_t stream) {
    const int rows = c0.n_rows + c1.n_rows;
    if (rows <= 0) return DAF_OK;
    cudaError_t e = launch_kernel(attn_combine_kernel, dim3((unsigned)((rows + 7) / 8)), dim3(256), 0, stream,
                                  /*after_kernel=*/true, c0, c1);
    count_launch();
    if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
    return check_launch();
}

int launch_attention(const void* q, const void* k, const void* v, int n_q, int n_kv, int Hq, int Hkv, int causal_off,
                     float scale, bool pack_group, bool allow_split, void* out, long long out_row_stride_bytes,
                     const int32_t* dst_rows, float* lse, DeviceStatus* status, void* scratch, size_t scratch_bytes,
                     cudaStream_t stream, bool after_kernel, const int32_t* q_pos) {
    if (n_q <= 0) return DAF_OK;
    const int G = Hq / Hkv;
    AttnPlan pl = plan_attention(n_q, n_kv, Hq, G, causal_off, pack_group, allow_split);
    const size_t need = attn_partial_bytes(n_q, Hq, pl.n_splits);
    if (need > scratch_bytes) return DAF_ERR_WORKSPACE;

    CUtensorMap tq, tk, tv;
    if (int rc = make_tmap(&tq, q, n_q, Hq, pl.Gp, pl.Tt)) return rc;
    if (int rc = make_tmap(&tk, k, n_kv, Hkv, 1, kSubN)) return rc;
    if (int rc = make_tmap(&tv, v, n_kv, Hkv, 1, kSubN)) return rc;
    // rows in token order leave by tiled stores: the output as a [n_q, Hq, 128] tensor with the caller's row stride
    const bool out_tiled = dst_rows == nullptr;
    CUtensorMap to = tq;
    if (out_tiled)
        if (int rc = make_tmap(&to, out, n_q, Hq, pl.Gp, pl.Tt, out_row_stride_bytes)) return rc;
    if (int rc = set_kernel_attributes()) return rc;

    AttnArgs a;
    memset(&a, 0, sizeof(a));
    SegArgs& s = a.seg[0];
    fill_problem(&s, n_q, n_kv, Hq, G, pl.Gp, causal_off, q_pos, scale, out, out_row_stride_bytes, dst_rows, lse);
    s.out_tiled = out_tiled ? 1 : 0;
    s.n_units = pl.n_tb;
    s.n_splits = pl.n_splits; s.tiles_per_split = pl.tiles_per_split;
    s.chunk = 0; s.n_slots = 0;
    s.n_items = pl.head_blocks * pl.n_tb * pl.n_splits;
    s.part_o = reinterpret_cast<float*>(scratch);
    s.part_lse = pl.n_splits > 1 ? reinterpret_cast<float*>(reinterpret_cast<char*>(scratch) +
                                                            (size_t)pl.n_splits * n_q * Hq * kD * sizeof(float))
                                 : nullptr;
    a.joint = 0;
    a.status = status;
    dim3 grid((unsigned)pl.head_blocks, (unsigned)pl.n_tb, (unsigned)pl.n_splits);
    cudaError_t e = launch_kernel(attn_fwd_kernel<false>, grid, dim3(kAttnThreads), kAttnSmemBytes, stream, after_kernel, tq, tk, tv, tq, tk, tv,
                                  to, to, a);
    count_launch();
    if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
    if (int rc = check_launch()) return rc;
    if (pl.n_splits > 1) {
        CombineSeg c0, c1;
        fill_combine(&c0, s);
        memset(&c1, 0, sizeof(c1));
        return launch_combine(c0, c1, stream);
    }
    return DAF_OK;
}

// Self-test of the bounded wait every kernel here relies on: two warps wait on a barrier that nothing ever
// signals.  The wait has to give up within `limit_ns`, record DAF_ERR_TIMEOUT and let the CTA return.
__global__ void __launch_bounds__(64)
bounded_wait_selftest_kernel(DeviceStatus* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    mbar_wait(&bar, 0, &abort_flag, status, 900, limit_ns);
}

int launch_bounded_wait_selftest(DeviceStatus* status, int limit_ms, cudaStream_t stream) {
    bounded_wait_selftest_kernel<<<1, 64, 0, stream>>>(status, (unsigned long long)limit_ms * 1000000ull);
    count_launch();
    return check_launch();
}

size_t joint_partial_bytes(const JointPlan& jp) { return jp.part_bytes_q + jp.part_bytes_i; }

int launch_attention_joint(const void* q_imp, const void* q_fresh, const int32_t* idx, const void* k_imp, const void* v_imp,
                           const void* k_fresh, const void* v_fresh,
                           int k, void* out_imp, const int32_t* dst_rows_imp, const void* q_question, const void* kv_k,
                           const void* kv_v,
                           int L_q, int L_d, void* out_question, long long out_row_stride_bytes, int Hq, int Hkv,
                           float scale, DeviceStatus* status, void* scratch, size_t scratch_bytes, cudaStream_t stream,
                           bool after_kernel, int launches) {
    const int G = Hq / Hkv, N = L_d + L_q;
    const JointPlan jp = plan_joint(k, L_q, L_d, Hq, G);
    if (joint_partial_bytes(jp) > scratch_bytes) return DAF_ERR_WORKSPACE;

    CUtensorMap tq0, tk0, tv0, tq1, tk1, tv1;
    // without packed Q rows the kernel reads them in place through idx (no tensor map needed for them)
    const bool gather_q = q_imp == nullptr;
    if (gather_q && (q_fresh == nullptr || idx == nullptr)) return DAF_ERR_INVALID_ARG;
    if (int rc = make_tmap(&tq0, gather_q ? q_question : q_imp, gather_q ? L_q : k, Hq, 1, kBlockM)) return rc;
    // without packed K/V rows the producer warp reads them in place through idx as well
    const bool gather_kv = k_imp == nullptr;
    if (gather_kv && (v_imp != nullptr || k_fresh == nullptr || v_fresh == nullptr || idx == nullptr)) return DAF_ERR_INVALID_ARG;
    if (!gather_kv && v_imp == nullptr) return DAF_ERR_INVALID_ARG;
    if (int rc = make_tmap(&tq1, q_question, L_q, Hq, jp.Gp_q, jp.Tt_q)) return rc;
    if (int rc = make_tmap(&tk1, kv_k, N, Hkv, 1, kSubN)) return rc;
    if (int rc = make_tmap(&tv1, kv_v, N, Hkv, 1, kSubN)) return rc;
    tk0 = tk1; tv0 = tv1;      // placeholders when the important rows' K/V are read in place
    if (!gather_kv) {
        if (int rc = make_tmap(&tk0, k_imp, k, Hkv, 1, kSubN)) return rc;
        if (int rc = make_tmap(&tv0, v_imp, k, Hkv, 1, kSubN)) return rc;
    }
    // final rows in token order (the compact layout) leave by tiled stores
    CUtensorMap to0 = tq1, to1 = tq1;
    const bool imp_tiled = dst_rows_imp == nullptr;
    if (imp_tiled)
        if (int rc = make_tmap(&to0, out_imp, k, Hq, 1, kBlockM, out_row_stride_bytes)) return rc;
    if (int rc = make_tmap(&to1, out_question, L_q, Hq, jp.Gp_q, jp.Tt_q, out_row_stride_bytes)) return rc;
    if (int rc = set_kernel_attributes()) return rc;

    AttnArgs a;
    memset(&a, 0, sizeof(a));
    char* sc = reinterpret_cast<char*>(scratch);
    // question rows: every unit cut into the same KV splits
    SegArgs& sq = a.seg[1];
    fill_problem(&sq, L_q, N, Hq, G, jp.Gp_q, L_d, nullptr, scale, out_question, out_row_stride_bytes, nullptr, nullptr);
    sq.out_tiled = 1;
    sq.n_units = jp.n_tb_q;
    sq.n_splits = jp.n_splits_q; sq.tiles_per_split = jp.tiles_per_split_q;
    sq.chunk = 0; sq.n_slots = 0;
    sq.n_items = jp.items_q;
    sq.part_o = reinterpret_cast<float*>(sc);
    sq.part_lse = reinterpret_cast<float*>(sc + (size_t)jp.n_splits_q * L_q * Hq * kD * sizeof(float));
    // important tokens: packed causal attention, long chains cut into balanced ranges
    SegArgs& si = a.seg[0];
    fill_problem(&si, k, k, Hq, G, 1, 0, nullptr, scale, out_imp, out_row_stride_bytes, dst_rows_imp, nullptr);
    if (gather_q) {
        si.q_src = reinterpret_cast<const __nv_bfloat16*>(q_fresh);
        si.q_idx = idx;
        si.q_src_rows = L_d;
    }
    if (gather_kv) {
        si.k_src = reinterpret_cast<const __nv_bfloat16*>(k_fresh);
        si.v_src = reinterpret_cast<const __nv_bfloat16*>(v_fresh);
        si.kv_idx = idx;
        si.kv_src_rows = L_d;
        si.kv_heads = Hkv;
    }
    si.out_tiled = imp_tiled ? 1 : 0;
    si.n_units = jp.n_tb_i;
    si.n_splits = 1; si.tiles_per_split = jp.n_tb_i;
    si.chunk = jp.chunk; si.n_slots = jp.n_slots;
    si.n_items = jp.items_i;
    const size_t rows_i = (size_t)jp.n_slots * kBlockM * Hq;
    si.part_o = reinterpret_cast<float*>(sc + jp.part_bytes_q);
    si.part_lse = reinterpret_cast<float*>(sc + jp.part_bytes_q + rows_i * kD * sizeof(float));
    a.joint = 1;
    a.status = status;

    const int items = jp.items_q + jp.items_i;
    if (launches & 1) {
        const cudaError_t e = gather_kv
            ? launch_kernel(attn_fwd_kernel<true>, dim3((unsigned)items), dim3(kAttnThreadsGather), kAttnSmemBytes, stream,
                            after_kernel, tq0, tk0, tv0, tq1, tk1, tv1, to0, to1, a)
            : launch_kernel(attn_fwd_kernel<false>, dim3((unsigned)items), dim3(kAttnThreads), kAttnSmemBytes, stream,
                            after_kernel, tq0, tk0, tv0, tq1, tk1, tv1, to0, to1, a);
        count_launch();
        if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
        if (int rc = check_launch()) return rc;
    }
    if (!(launches & 2)) return DAF_OK;
    CombineSeg ci, cq;
    fill_combine(&ci, si);
    fill_combine(&cq, sq);
    return launch_combine(ci, cq, stream);
}

}  // namespace daf

// ------------------------------------------------------------------------------------------------
// Allocation-free question-document attention.
//
// Some callers hold every byte of device memory themselves and cannot ask the
// driver for more at the moment they need this step: a serving loop whose memory
// pool has already claimed the whole GPU, a plug-in running inside another
// framework's allocator where a driver allocation would stall the device, or a
// latency-critical path where an allocation's implicit synchronisation is not
// acceptable.  For them the split-KV partial results and the status word of the
// question-document stage live in the fixed device array below instead of a
// caller-provided workspace.  Every GPU that loads this library carries the array
// until the process exits.
namespace {
constexpr size_t kStaticScratchBytes = (size_t)16 << 20;   // 16 MiB: status word + split-KV partials
static __device__ __align__(256) unsigned char g_qd_static_scratch[kStaticScratchBytes];
constexpr int kMaxDevices = 64;
// one slot per device; concurrent first calls on a device resolve the same address and store the same value
std::atomic<void*> g_static_scratch_addr[kMaxDevices];

// In host code the array's name is only a handle for the runtime, not an address
// a kernel can use, so the device address is looked up once per device.
int static_scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { daf::set_cuda_error(e); return DAF_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return DAF_ERR_UNSUPPORTED;
    void* known = g_static_scratch_addr[dev].load(std::memory_order_acquire);
    if (known == nullptr) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_qd_static_scratch);
        if (e != cudaSuccess || ptr == nullptr) {
            daf::set_cuda_error(e != cudaSuccess ? e : cudaErrorInvalidSymbol);
            return DAF_ERR_CUDA;
        }
        g_static_scratch_addr[dev].store(ptr, std::memory_order_release);
        known = ptr;
    }
    *out = known;
    return DAF_OK;
}
}  // namespace

extern "C" size_t daf_qd_attn_static_max_bytes(void) { return kStaticScratchBytes; }

extern "C" int daf_qd_attn_static(const daf_params* p, const void* q_question, const void* kv_k, const void* kv_v,
                                  void* out, int64_t out_row_stride_bytes, const int32_t* dst_rows, float* lse,
                                  void* stream) {
    using namespace daf;
    ResolvedParams rp;
    if (int rc = resolve_params(p, &rp)) return rc;
    if (rp.L_q == 0) return DAF_OK;
    if (!q_question || !kv_k || !kv_v || !out) return DAF_ERR_INVALID_ARG;
    if (!aligned16(q_question) || !aligned16(kv_k) || !aligned16(kv_v) || !aligned16(out) ||
        out_row_stride_bytes % 16 != 0) return DAF_ERR_ALIGNMENT;
    if (out_row_stride_bytes < (int64_t)rp.Hq * 256) return DAF_ERR_INVALID_ARG;
    // the fixed array must hold the status word and this problem's split-KV partials
    const AttnPlan pl = plan_attention(rp.L_q, rp.N, rp.Hq, rp.G, rp.L_d, true, true);
    const size_t need = kStatusBytes + attn_partial_bytes(rp.L_q, rp.Hq, pl.n_splits);
    if (need > kStaticScratchBytes) return DAF_ERR_WORKSPACE;   // problem too large for the fixed scratch
    void* base = nullptr;
    if (int rc = static_scratch_address(&base)) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the status word has to start at zero
    cudaError_t e = cudaMemsetAsync(base, 0, kStatusBytes, st);
    if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
    return launch_attention(q_question, kv_k, kv_v, rp.L_q, rp.N, rp.Hq, rp.Hkv, rp.L_d, rp.scale, true, true, out,
                            out_row_stride_bytes, dst_rows, lse, reinterpret_cast<DeviceStatus*>(base),
                            reinterpret_cast<char*>(base) + kStatusBytes, kStaticScratchBytes - kStatusBytes, st);
}

// Status of the calls made through daf_qd_attn_static on the current device since the last poll: the
// status word sits at the head of the fixed array, so it is read (and cleared) from there.  No allocation.
extern "C" int daf_qd_attn_static_poll_status(void* stream) {
    using namespace daf;
    void* base = nullptr;
    if (int rc = static_scratch_address(&base)) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    DeviceStatus hs;
    cudaError_t e = cudaMemcpyAsync(&hs, base, sizeof(hs), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e == cudaSuccess && hs.code != 0) {
        e = cudaMemsetAsync(base, 0, sizeof(hs), st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    }
    if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
    return hs.code;
}
