// Step 1 of the DAF layer (Methods, item 1 "selection" and "gather"; item 2
// "hybrid KV cache") and the stand-alone form of step 4 (item 3 "state fusion").
//
// These steps move bytes and rank 32-bit keys; they are bound by HBM bandwidth
// and launch latency, not by arithmetic, so they are plain coalesced 16-byte
// kernels with no tensor-core work.
#include <cooperative_groups.h>
#include <cuda_fp8.h>

#include <atomic>

#include "daf_common.cuh"

namespace daf {

#ifdef DAF_TRACE
DAF_KT_TABLE;
DAF_KT_READER(daf_dbg_kt_select)
#endif

// ------------------------------------------------------------------ selection
// A cluster of 8 CTAs ranks all L_d aggregated scores.  Each CTA keeps a
// contiguous slice of the keys in its shared memory.  Four passes of an
// 8-bit radix select find the key of the k-th largest score: every CTA builds
// a 256-bin histogram of its slice, the histograms are summed through
// distributed shared memory, and every CTA picks the same digit.  An ordered
// compaction then emits the selected positions in ascending order.  Ties at
// the threshold are broken by position (lower first), so the result is unique.

constexpr int kSelCluster = 8;
constexpr int kSelThreads = 512;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelSmemKeysPerCta = 40960;   // slice kept in shared memory up to this size, in global scratch beyond

// Monotone map fp32 -> uint32: larger score <=> larger key; -0 == +0; NaN -> 0 (ranks lowest).
__device__ __forceinline__ uint32_t score_key(float s) {
    uint32_t b = __float_as_uint(s);
    if ((b & 0x7FFFFFFFu) > 0x7F800000u) return 0u;   // NaN
    if (b == 0x80000000u) b = 0u;                     // -0 -> +0
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// fp32 add, round to nearest, subnormals kept (the library is built with flush-to-zero arithmetic; the
// aggregation of the signal rows must not flush, or tiny sums would all rank as ties at zero).
__device__ __forceinline__ float add_rn_keep_subnormals(float a, float b) {
    float d;
    asm("add.rn.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

// Keys sit in shared memory with one word of padding per 32, so that both access patterns are free of bank
// conflicts: consecutive threads reading consecutive keys, and each thread walking its own run of keys.
__host__ __device__ __forceinline__ int padded(int i) { return i + (i >> 5); }

struct SelShared {
    uint32_t hist[2][256];     // double-buffered so that a peer may still read pass p while pass p+1 is filled
    uint32_t total[256];
    uint32_t scan_gt[kSelWarps];
    uint32_t scan_eq[kSelWarps];
    uint32_t cta_counts[2];    // this CTA's number of keys above / equal to the threshold (read by peers)
    uint32_t pick[3];          // chosen prefix, remaining rank, number of keys in the chosen bin
};

__global__ void __cluster_dims__(kSelCluster, 1, 1) __launch_bounds__(kSelThreads, 1)
select_topk_kernel(const float* __restrict__ scores, int n_sig, int L_d, int k,
                   uint32_t* __restrict__ gkeys, int32_t* __restrict__ idx_out, int wait_at_end) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    DAF_KT_BEGIN(0);
    // The kernel launched just before this one is either the one that wrote the scores (wait for it now) or one
    // this kernel does not depend on (the expansion of an fp8 cache: run beside it and wait for it only at the
    // end, so that the kernel behind this one finds both finished).
    if (!wait_at_end) pdl_wait();
    pdl_launch_dependents();   // the gather kernel may start launching; it waits for this grid before reading idx
    extern __shared__ __align__(16) unsigned char sel_smem[];
    SelShared* sh = reinterpret_cast<SelShared*>(sel_smem);
    uint32_t* skeys = reinterpret_cast<uint32_t*>(sel_smem + sizeof(SelShared));

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rank = (int)cluster.block_rank();
    const int per_cta = (L_d + kSelCluster - 1) / kSelCluster;
    const int lo_cta = min(L_d, rank * per_cta);
    const int n_loc = min(L_d, lo_cta + per_cta) - lo_cta;
    const bool in_smem = per_cta <= kSelSmemKeysPerCta;
    uint32_t* keys = in_smem ? skeys : (gkeys + lo_cta);
    auto at = [&](int i) { return in_smem ? padded(i) : i; };   // padded layout in shared memory only

    // aggregate the signal rows in ascending row order (fp32 adds, no fusing) and build keys
    for (int i = tid; i < n_loc; i += kSelThreads) {
        const int g = lo_cta + i;
        float acc = scores[g];
        for (int l = 1; l < n_sig; ++l) acc = add_rn_keep_subnormals(acc, scores[(size_t)l * L_d + g]);
        keys[at(i)] = score_key(acc);
    }
    if (tid < 256) { sh->hist[0][tid] = 0u; sh->hist[1][tid] = 0u; }
    if (tid == 0) { sh->pick[0] = 0u; sh->pick[1] = (uint32_t)k; sh->pick[2] = 0u; }
    __syncthreads();

    // Radix selection from the top byte down.  It stops as soon as every key left in the chosen bin is taken
    // (with distinct scores usually after three passes): the comparisons below then look only at the bits
    // resolved so far.
    uint32_t prefix = 0u, mask = 0u;
    int pass = 0;
    for (int shift = 24; shift >= 0; shift -= 8, ++pass) {
        uint32_t* hist = sh->hist[pass & 1];
        const int n_round = (n_loc + 31) / 32 * 32;
        for (int i = tid; i < n_round; i += kSelThreads) {
            bool in = false;
            uint32_t bin = 0u;
            if (i < n_loc) {
                const uint32_t key = keys[at(i)];
                in = (key & mask) == prefix;
                bin = (key >> shift) & 0xFFu;
            }
            // a warp whose keys all fall in one bin adds once; otherwise every thread adds for itself
            const uint32_t active = __ballot_sync(0xFFFFFFFFu, in);
            if (active == 0u) continue;
            const uint32_t lead_bin = __shfl_sync(0xFFFFFFFFu, bin, __ffs(active) - 1);
            const uint32_t same = __ballot_sync(0xFFFFFFFFu, in && bin == lead_bin);
            if (same == active) {
                if (lane == __ffs(active) - 1) atomicAdd(&hist[lead_bin], (uint32_t)__popc(active));
            } else if (in) {
                atomicAdd(&hist[bin], 1u);
            }
        }
        cluster.sync();   // every CTA's histogram of this pass is complete
        if (tid < 256) {
            uint32_t sum = 0;
#pragma unroll
            for (int r = 0; r < kSelCluster; ++r) sum += cluster.map_shared_rank(hist, r)[tid];
            sh->total[tid] = sum;
            sh->hist[(pass + 1) & 1][tid] = 0u;   // peers finished reading this buffer two syncs ago
        }
        __syncthreads();
        if (warp == 0) {
            // lane l owns bins [8*(31-l), 8*(31-l)+7]; lane 0 holds the highest bins
            const int base = 8 * (31 - lane);
            uint32_t sgrp = 0;
            for (int b = 0; b < 8; ++b) sgrp += sh->total[base + b];
            uint32_t incl = sgrp;
            for (int o = 1; o < 32; o <<= 1) {
                uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += t;
            }
            const uint32_t above = incl - sgrp;
            const uint32_t k_rem = sh->pick[1];
            __syncwarp();   // every lane has read the rank before one of them replaces it
            if (k_rem > above && k_rem <= incl) {
                uint32_t a = above;
                for (int b = 7; b >= 0; --b) {
                    const uint32_t c = sh->total[base + b];
                    if (k_rem <= a + c) {
                        sh->pick[0] = prefix | ((uint32_t)(base + b) << shift);
                        sh->pick[1] = k_rem - a;
                        sh->pick[2] = c;
                        break;
                    }
                    a += c;
                }
            }
        }
        __syncthreads();
        prefix = sh->pick[0];
        mask |= 0xFFu << shift;
        if (sh->pick[2] == sh->pick[1]) break;   // every key left in the bin is taken: no need to tell them apart
    }
    const uint32_t thr = prefix;           // the resolved bits of the k-th largest key
    const uint32_t need_eq = sh->pick[1];  // how many keys matching thr are taken (lowest positions first)

    // ordered compaction: thread t owns the contiguous local positions [t*E, (t+1)*E)
    const int E = (per_cta + kSelThreads - 1) / kSelThreads;
    const int lo = min(n_loc, tid * E), hi = min(n_loc, lo + E);
    uint32_t n_gt = 0, n_eq = 0;
    for (int i = lo; i < hi; ++i) {
        const uint32_t key = keys[at(i)] & mask;
        n_gt += key > thr;
        n_eq += key == thr;
    }
    uint32_t in_gt = n_gt, in_eq = n_eq;
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t a = __shfl_up_sync(0xFFFFFFFFu, in_gt, o), b = __shfl_up_sync(0xFFFFFFFFu, in_eq, o);
        if (lane >= o) { in_gt += a; in_eq += b; }
    }
    if (lane == 31) { sh->scan_gt[warp] = in_gt; sh->scan_eq[warp] = in_eq; }
    __syncthreads();
    if (warp == 0) {
        uint32_t a = lane < kSelWarps ? sh->scan_gt[lane] : 0u, b = lane < kSelWarps ? sh->scan_eq[lane] : 0u;
        uint32_t ia = a, ib = b;
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t x = __shfl_up_sync(0xFFFFFFFFu, ia, o), y = __shfl_up_sync(0xFFFFFFFFu, ib, o);
            if (lane >= o) { ia += x; ib += y; }
        }
        if (lane < kSelWarps) { sh->scan_gt[lane] = ia - a; sh->scan_eq[lane] = ib - b; }
        if (lane == kSelWarps - 1) { sh->cta_counts[0] = ia; sh->cta_counts[1] = ib; }
    }
    cluster.sync();   // every CTA's counts are visible
    uint32_t gt_before = sh->scan_gt[warp] + in_gt - n_gt;
    uint32_t eq_before = sh->scan_eq[warp] + in_eq - n_eq;
    for (int r = 0; r < rank; ++r) {
        const uint32_t* c = cluster.map_shared_rank(sh->cta_counts, r);
        gt_before += c[0];
        eq_before += c[1];
    }
    if (k > 0) {
        uint32_t pos = gt_before + min(eq_before, need_eq);
        for (int i = lo; i < hi; ++i) {
            const uint32_t key = keys[at(i)] & mask;
            bool take = key > thr;
            if (key == thr) { take = eq_before < need_eq; ++eq_before; }
            if (take) idx_out[pos++] = lo_cta + i;
        }
    }
    cluster.sync();   // no CTA may retire while a peer can still read its shared memory
    if (wait_at_end) pdl_wait();
    DAF_KT_END(0);
}

// ------------------------------------------------ selection, one CTA (up to 16K tokens)
// Latency matters more than bandwidth here (at most 64 KB of keys), so the common sizes run in one
// CTA with no cluster traffic.  The keys are first reduced to their offset from the smallest key.  One
// pass over all keys histograms the top 11 of the bits that offset needs (typically 24-27 of 32, fewer
// when the scores are close together) with shared-memory atomics and finds the bin that holds the k-th
// largest key; only the keys of that bin (typically well under one per cent) go on: when they are few,
// each is ranked against the others directly, otherwise passes of 9 bits fix the remaining bits.  Because the offsets of real scores spread over the whole histogram,
// the atomics rarely collide; scores that are all (nearly) equal collide more, and all of them become
// candidates, but the result stays correct.  An ordered compaction then emits the positions.
constexpr int kSel1Threads = 1024;
constexpr int kSel1Warps = kSel1Threads / 32;
constexpr int kSel1MaxKeys = 16384;   // capacity of the one-CTA kernel (keys live in shared memory)
constexpr int kSel1TopBits = 11;      // first pass, over all keys
constexpr int kSel1TopBins = 1 << kSel1TopBits;
constexpr int kSel1Bits = 9;          // later passes, over the candidates
constexpr int kSel1Bins = 1 << kSel1Bits;

struct Sel1Shared {
    uint32_t hist[kSel1TopBins];
    uint32_t warp_a[kSel1Warps];
    uint32_t warp_b[kSel1Warps];
    uint32_t pick[2];       // chosen digit, remaining rank
    uint32_t n_cand;
};

// Exclusive prefix sums of (a, b) over the threads of the CTA, in thread order.
__device__ __forceinline__ void block_excl_scan2(uint32_t a, uint32_t b, uint32_t* wa, uint32_t* wb,
                                                 uint32_t& ex_a, uint32_t& ex_b, uint32_t& tot_a, uint32_t& tot_b) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t ia = a, ib = b;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t x = __shfl_up_sync(0xFFFFFFFFu, ia, o), y = __shfl_up_sync(0xFFFFFFFFu, ib, o);
        if (lane >= o) { ia += x; ib += y; }
    }
    if (lane == 31) { wa[warp] = ia; wb[warp] = ib; }
    __syncthreads();
    uint32_t va = wa[lane], vb = wb[lane];   // kSel1Warps == 32: one warp total per lane
    uint32_t sa = va, sb = vb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t x = __shfl_up_sync(0xFFFFFFFFu, sa, o), y = __shfl_up_sync(0xFFFFFFFFu, sb, o);
        if (lane >= o) { sa += x; sb += y; }
    }
    tot_a = __shfl_sync(0xFFFFFFFFu, sa, 31);
    tot_b = __shfl_sync(0xFFFFFFFFu, sb, 31);
    ex_a = __shfl_sync(0xFFFFFFFFu, sa - va, warp) + ia - a;
    ex_b = __shfl_sync(0xFFFFFFFFu, sb - vb, warp) + ib - b;
    __syncthreads();   // wa/wb may be reused by the next scan
}

// Finds, from the top, the bin in which the k_rem-th element falls.  Thread t owns `per` consecutive
// bins in descending order; the result goes to pick[0] (bin) and pick[1] (rank inside that bin).
__device__ __forceinline__ void pick_bin(Sel1Shared* sh, int n_bins, int per) {
    const int top = n_bins - 1 - (int)threadIdx.x * per;   // this thread's highest bin
    // the remaining rank is read here, ahead of the scan: the scan's barriers then separate every
    // thread's read from the one thread that writes the reduced rank below
    const uint32_t k_rem = sh->pick[1];
    uint32_t c = 0;
    if (top >= 0)
        for (int b = 0; b < per; ++b) c += sh->hist[top - b];
    uint32_t above, dummy, tot, tot2;
    block_excl_scan2(c, 0u, sh->warp_a, sh->warp_b, above, dummy, tot, tot2);
    if (top >= 0 && k_rem > above && k_rem <= above + c) {
        uint32_t acc = above;
        for (int b = 0; b < per; ++b) {
            const uint32_t cb = sh->hist[top - b];
            if (k_rem <= acc + cb) { sh->pick[0] = (uint32_t)(top - b); sh->pick[1] = k_rem - acc; break; }
            acc += cb;
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kSel1Threads, 1)
select_topk_cta_kernel(const float* __restrict__ scores, int n_sig, int L_d, int k, int32_t* __restrict__ idx_out,
                       int wait_at_end) {
    extern __shared__ __align__(16) unsigned char sel_smem[];
    Sel1Shared* sh = reinterpret_cast<Sel1Shared*>(sel_smem);
    uint32_t* keys = reinterpret_cast<uint32_t*>(sel_smem + sizeof(Sel1Shared));
    uint32_t* cand = keys + padded(L_d);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    DAF_KT_BEGIN(0);
    if (!wait_at_end) pdl_wait();   // see select_topk_kernel
    pdl_launch_dependents();   // the gather kernel may start launching; it waits for this grid before reading idx

    // aggregate the signal rows in ascending row order (fp32 adds, no fusing), build keys, find their range
    // (eight loads in flight per thread: one load per trip would serialise on memory latency)
    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
    for (int base = tid; base < L_d; base += 8 * kSel1Threads) {
        float acc[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = base + u * kSel1Threads;
            acc[u] = i < L_d ? scores[i] : 0.f;
        }
        for (int l = 1; l < n_sig; ++l) {
            float nxt[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = base + u * kSel1Threads;
                nxt[u] = i < L_d ? scores[(size_t)l * L_d + i] : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) acc[u] = add_rn_keep_subnormals(acc[u], nxt[u]);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = base + u * kSel1Threads;
            if (i < L_d) {
                const uint32_t key = score_key(acc[u]);
                keys[padded(i)] = key;
                kmin = min(kmin, key);
                kmax = max(kmax, key);
            }
        }
    }
    for (int i = tid; i < kSel1TopBins; i += kSel1Threads) sh->hist[i] = 0u;
    if (tid == 0) { sh->pick[0] = 0u; sh->pick[1] = (uint32_t)k; sh->n_cand = 0u; }
    kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
    kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
    if (lane == 0) { sh->warp_a[warp] = kmin; sh->warp_b[warp] = kmax; }
    __syncthreads();
    kmin = __reduce_min_sync(0xFFFFFFFFu, sh->warp_a[lane]);
    kmax = __reduce_max_sync(0xFFFFFFFFu, sh->warp_b[lane]);
    __syncthreads();   // warp_a/warp_b are reused by the scans below
    const uint32_t range = kmax - kmin;
    const int bits = 32 - __clz((int)range);        // bits the offsets need (0 when all keys are equal)
    const int low_bits = max(bits - kSel1TopBits, 0);   // bits left after the first pass

    // first pass, all keys: the top bits of the offset
    for (int i = tid; i < L_d; i += kSel1Threads) atomicAdd(&sh->hist[(keys[padded(i)] - kmin) >> low_bits], 1u);
    __syncthreads();
    pick_bin(sh, kSel1TopBins, kSel1TopBins / kSel1Threads);
    const uint32_t top_digit = sh->pick[0];
    // candidates: the low bits of the keys that fall in the chosen bin
    for (int i = tid; i < L_d; i += kSel1Threads) {
        const uint32_t off = keys[padded(i)] - kmin;
        if ((off >> low_bits) == top_digit) cand[atomicAdd(&sh->n_cand, 1u)] = low_bits > 0 ? off & ((1u << low_bits) - 1u) : 0u;
    }
    if (tid < kSel1Bins) sh->hist[tid] = 0u;
    __syncthreads();
    const int n_cand = (int)sh->n_cand;    // at most L_d, the capacity of the list
    int passes = (low_bits + kSel1Bits - 1) / kSel1Bits;
    uint32_t prefix = 0u;      // the low digits fixed so far
    if (passes > 0 && n_cand <= kSel1Threads) {
        // few candidates (the usual case): each thread ranks one candidate by counting the larger and the
        // equal ones; the candidate whose rank interval holds the remaining rank is the threshold
        const uint32_t k_rem = sh->pick[1];
        __syncthreads();   // every thread has read the rank before one of them replaces it
        if (tid < n_cand) {
            const uint32_t mine = cand[tid];
            uint32_t n_gt = 0, n_eq = 0;
            for (int j = 0; j < n_cand; ++j) {
                const uint32_t other = cand[j];
                n_gt += other > mine;
                n_eq += other == mine;
            }
            if (k_rem > n_gt && k_rem <= n_gt + n_eq) { sh->pick[0] = mine; sh->pick[1] = k_rem - n_gt; }   // equal candidates write the same
        }
        __syncthreads();
        prefix = sh->pick[0];
        passes = 0;
    }
    for (int p = 0; p < passes; ++p) {
        const int shift = (passes - 1 - p) * kSel1Bits;
        for (int i = tid; i < n_cand; i += kSel1Threads) {
            const uint32_t low = cand[i];
            if ((low >> (shift + kSel1Bits)) == prefix) atomicAdd(&sh->hist[(low >> shift) & (kSel1Bins - 1)], 1u);
        }
        __syncthreads();
        pick_bin(sh, kSel1Bins, 1);
        prefix = (prefix << kSel1Bits) | sh->pick[0];
        if (tid < kSel1Bins) sh->hist[tid] = 0u;
        __syncthreads();
    }
    prefix |= top_digit << low_bits;       // the whole offset of the threshold (passes == 0: the top digit alone)
    const uint32_t thr = kmin + prefix;    // key of the k-th largest score (passes == 0: every key equals kmin)
    const uint32_t need_eq = sh->pick[1];  // how many keys equal to thr are taken (lowest positions first)

    // ordered compaction: thread t owns the contiguous positions [t*E, (t+1)*E)
    const int E = (L_d + kSel1Threads - 1) / kSel1Threads;
    const int lo = min(L_d, tid * E), hi = min(L_d, lo + E);
    uint32_t n_gt = 0, n_eq = 0;
    for (int i = lo; i < hi; ++i) {
        const uint32_t key = keys[padded(i)];
        n_gt += key > thr;
        n_eq += key == thr;
    }
    uint32_t gt_before, eq_before, tot_gt, tot_eq;
    block_excl_scan2(n_gt, n_eq, sh->warp_a, sh->warp_b, gt_before, eq_before, tot_gt, tot_eq);
    if (k > 0) {
        uint32_t pos = gt_before + min(eq_before, need_eq);
        for (int i = lo; i < hi; ++i) {
            const uint32_t key = keys[padded(i)];
            bool take = key > thr;
            if (key == thr) { take = eq_before < need_eq; ++eq_before; }
            if (take) idx_out[pos++] = i;
        }
    }
    if (wait_at_end) pdl_wait();
    DAF_KT_END(0);
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

// kFar: the fresh rows come from far away (pinned host memory, read over the host link): every thread requests all
// its chunks of the row before it stores any, so that one round trip covers them.  For rows in device memory the
// plain loop is the faster one inside a layer (the batched form made the layer 0.4 us slower at 16k).
constexpr int kRowMaxChunks = 4;      // 4 x 192 x 16 B = 12 KB: a row of 32 + 2 x 8 heads
template <bool kFar>
__global__ void __launch_bounds__(kRowThreads)
gather_update_kernel(const GatherArgs a) {
    DAF_KT_BEGIN(1);
    pdl_wait();                // idx may come from the selection kernel launched just before; the packed buffers may still be read by the previous layer
    DAF_KT_BEGIN(2);
    pdl_launch_dependents();   // the attention kernel may start launching; it waits for this grid
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
        // no packed Q wanted: K, V only; no packed K/V wanted and nothing to overwrite in the cache: nothing at all
        const int c_end = (a.k_pack != nullptr || a.overwrite) ? per_row : a.cq;
        const int c0 = (a.q_pack != nullptr ? 0 : a.cq) + threadIdx.x;
        if (kFar) {
            for (int base = c0; base < c_end; base += kRowThreads * kRowMaxChunks) {
                int4 v[kRowMaxChunks];
#pragma unroll
                for (int u = 0; u < kRowMaxChunks; ++u) {
                    const int c = base + u * kRowThreads;
                    if (c < a.cq) v[u] = __ldg(a.q_fresh + qsrc + c);
                    else if (c < a.cq + a.ckv) v[u] = __ldg(a.k_fresh + ksrc + (c - a.cq));
                    else if (c < c_end) v[u] = __ldg(a.v_fresh + ksrc + (c - a.cq - a.ckv));
                }
#pragma unroll
                for (int u = 0; u < kRowMaxChunks; ++u) {
                    const int c = base + u * kRowThreads;
                    if (c < a.cq) {
                        a.q_pack[qdst + c] = v[u];
                    } else if (c < a.cq + a.ckv) {
                        const int cc = c - a.cq;
                        if (a.k_pack != nullptr) a.k_pack[kdst + cc] = v[u];
                        if (a.overwrite) a.kv_k[ksrc + cc] = v[u];
                    } else if (c < c_end) {
                        const int cc = c - a.cq - a.ckv;
                        if (a.v_pack != nullptr) a.v_pack[kdst + cc] = v[u];
                        if (a.overwrite) a.kv_v[ksrc + cc] = v[u];
                    }
                }
            }
        } else {
            for (int c = c0; c < c_end; c += kRowThreads) {
                if (c < a.cq) {
                    a.q_pack[qdst + c] = __ldg(a.q_fresh + qsrc + c);
                } else if (c < a.cq + a.ckv) {
                    const int cc = c - a.cq;
                    const int4 v = __ldg(a.k_fresh + ksrc + cc);
                    if (a.k_pack != nullptr) a.k_pack[kdst + cc] = v;
                    if (a.overwrite) a.kv_k[ksrc + cc] = v;
                } else {
                    const int cc = c - a.cq - a.ckv;
                    const int4 v = __ldg(a.v_fresh + ksrc + cc);
                    if (a.v_pack != nullptr) a.v_pack[kdst + cc] = v;
                    if (a.overwrite) a.kv_v[ksrc + cc] = v;
                }
            }
        }
    } else {
        const size_t off = (size_t)(a.L_d + (row - a.k)) * a.ckv;
        for (int c = threadIdx.x; c < 2 * a.ckv; c += kRowThreads) {
            if (c < a.ckv) a.kv_k[off + c] = __ldg(a.k_fresh + off + c);
            else a.kv_v[off + c - a.ckv] = __ldg(a.v_fresh + off + c - a.ckv);
        }
    }
    DAF_KT_END(1);
}

// ------------------------------------------------------------- state fusion
struct FuseArgs {
    const int4* o_imp; const int4* o_q; int4* hidden;
    const int32_t* idx; int32_t* row_pos;
    int k, L_d, L_q, cq, mode;
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

// ------------------------------------------------------------ deviation signal
// Per-layer importance signal of a document token: squared deviation of its fresh K and V rows from
// the cached ones, summed over heads and channels (Methods, item 1; the formula is this library's
// reading).  A streaming reduction: one warp per token, 16-byte loads, fp32 accumulation, a fixed
// shuffle tree, so the result does not depend on the launch shape.
__device__ __forceinline__ float sq_dev8(const int4 a, const int4 b) {
    const __nv_bfloat162* x = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* y = reinterpret_cast<const __nv_bfloat162*>(&b);
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 fx = __bfloat1622float2(x[i]), fy = __bfloat1622float2(y[i]);
        const float d0 = fx.x - fy.x, d1 = fx.y - fy.y;
        acc = fmaf(d0, d0, acc);
        acc = fmaf(d1, d1, acc);
    }
    return acc;
}

__global__ void __launch_bounds__(256)
deviation_scores_kernel(const int4* __restrict__ k_fresh, const int4* __restrict__ v_fresh,
                        const int4* __restrict__ k_cached, const int4* __restrict__ v_cached,
                        int L_d, int chunks_per_row, float* __restrict__ scores) {
    const int lane = threadIdx.x & 31;
    const int warps_per_grid = (int)(gridDim.x * (blockDim.x >> 5));
    for (int tok = (int)(blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)); tok < L_d; tok += warps_per_grid) {
        const size_t base = (size_t)tok * chunks_per_row;
        float acc = 0.f;
        for (int c = lane; c < chunks_per_row; c += 32) {
            acc += sq_dev8(__ldg(k_fresh + base + c), __ldg(k_cached + base + c));
            acc += sq_dev8(__ldg(v_fresh + base + c), __ldg(v_cached + base + c));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) scores[tok] = acc;
    }
}

// The same signal for several layers at once, aggregated on the fly (Methods, item 1: the signals of several
// layers, typically the 2nd to 4th, are aggregated before the tokens are ranked).  One warp per token walks
// the signal layers in ascending order: each layer's value is computed exactly as deviation_scores_kernel
// computes it (same chunk order, same shuffle tree) and added to the running fp32 sum with a plain
// round-to-nearest add, subnormals kept -- the order and arithmetic in which the selection kernels
// aggregate the rows of a score matrix -- so ranking the sums gives the positions that the two-step route
// (one daf_deviation_scores call per layer, then daf_select on the [n_sig, L_d] matrix) would give, without
// that matrix ever being written.
constexpr int kMaxSignalLayers = 8;
struct SignalLayers {
    const int4* k_fresh[kMaxSignalLayers]; const int4* v_fresh[kMaxSignalLayers];
    const int4* k_cached[kMaxSignalLayers]; const int4* v_cached[kMaxSignalLayers];
    int n;
};

__global__ void __launch_bounds__(256)
deviation_sum_kernel(const SignalLayers layers, int L_d, int chunks_per_row, float* __restrict__ sums) {
    pdl_launch_dependents();   // the selection kernel may start launching; it waits for this grid before reading sums
    const int lane = threadIdx.x & 31;
    const int warps_per_grid = (int)(gridDim.x * (blockDim.x >> 5));
    for (int tok = (int)(blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)); tok < L_d; tok += warps_per_grid) {
        const size_t base = (size_t)tok * chunks_per_row;
        float total = 0.f;
        for (int l = 0; l < layers.n; ++l) {
            const int4* kf = layers.k_fresh[l]; const int4* vf = layers.v_fresh[l];
            const int4* kc = layers.k_cached[l]; const int4* vc = layers.v_cached[l];
            float acc = 0.f;
            for (int c = lane; c < chunks_per_row; c += 32) {
                acc += sq_dev8(__ldg(kf + base + c), __ldg(kc + base + c));
                acc += sq_dev8(__ldg(vf + base + c), __ldg(vc + base + c));
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
            total = l == 0 ? acc : add_rn_keep_subnormals(total, acc);
        }
        if (lane == 0) sums[tok] = total;
    }
}

// ----------------------------------------------------------------- host side
// Measured on B200 (selection alone): one CTA 4.9 / 5.3 / 8.1 us at 6K / 8K / 16K tokens, the cluster of eight
// 7.0 / 5.8 / 7.6 us: one CTA up to 8K tokens, the cluster beyond.
static int g_sel1_max_keys = 8192;
#ifdef DAF_TRACE
extern "C" void daf_dbg_sel1_max_keys(int n) { g_sel1_max_keys = n < kSel1MaxKeys ? n : kSel1MaxKeys; }
#endif

size_t select_scratch_bytes(int L_d) {
    const int per_cta = (L_d + kSelCluster - 1) / kSelCluster;
    return per_cta > kSelSmemKeysPerCta ? ((size_t)per_cta * kSelCluster * sizeof(uint32_t) + 255) / 256 * 256 : 0;
}

static size_t select_smem_bytes(int L_d) {
    const int per_cta = (L_d + kSelCluster - 1) / kSelCluster;
    return sizeof(SelShared) + (per_cta <= kSelSmemKeysPerCta ? (size_t)padded(per_cta) * sizeof(uint32_t) : 0);
}

int launch_select(const ResolvedParams& rp, const float* scores, int n_sig, const int32_t* idx_in,
                  const void* q_fresh, const void* k_fresh, const void* v_fresh, void* kv_k, void* kv_v,
                  int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack,
                  DeviceStatus* status, void* scratch, cudaStream_t stream, bool scores_from_previous_kernel,
                  bool beside_previous_kernel, bool select_only, bool rows_far) {
    // beside_previous_kernel: the kernel launched just before (the fp8 cache expansion) is independent of the
    // selection; the selection kernel starts while it runs and only waits for it before it retires
    const bool dependent = scores_from_previous_kernel || beside_previous_kernel;
    const int wait_at_end = beside_previous_kernel ? 1 : 0;
    const int32_t* idx_src = idx_in;
    if (scores != nullptr && rp.L_d > 0 && rp.k > 0) {
        static std::atomic<bool> attr_done[64];   // per device; a concurrent first call sets the same values
        int dev = 0;
        cudaGetDevice(&dev);
        if (dev >= 0 && dev < 64 && !attr_done[dev].load(std::memory_order_acquire)) {
            cudaError_t e = cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)(sizeof(SelShared) + (size_t)padded(kSelSmemKeysPerCta) * sizeof(uint32_t)));
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(select_topk_cta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(sizeof(Sel1Shared) + ((size_t)padded(kSel1MaxKeys) + kSel1MaxKeys) * sizeof(uint32_t)));
            if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
            attr_done[dev].store(true, std::memory_order_release);
        }
        if (rp.L_d <= g_sel1_max_keys) {
            const size_t smem1 = sizeof(Sel1Shared) + ((size_t)padded(rp.L_d) + rp.L_d) * sizeof(uint32_t);   // keys and candidate list
            const cudaError_t e = launch_kernel(select_topk_cta_kernel, dim3(1), dim3(kSel1Threads), smem1, stream,
                                                dependent, scores, n_sig, rp.L_d, rp.k, idx_out, wait_at_end);
            if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
        } else {
            const size_t smem = select_smem_bytes(rp.L_d);
            const cudaError_t e = launch_kernel(select_topk_kernel, dim3(kSelCluster), dim3(kSelThreads), smem, stream,
                                                dependent, scores, n_sig, rp.L_d, rp.k,
                                                reinterpret_cast<uint32_t*>(scratch), idx_out, wait_at_end);
            if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
        }
        count_launch();
        if (int rc = check_launch()) return rc;
        idx_src = idx_out;
    }
    const int rows = select_only ? 0 : rp.k + rp.L_q;
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
        // Always a programmatic dependent of whatever kernel precedes it on the stream: the kernel waits for that
        // kernel to complete before it touches anything (so the result is that of a plain launch), but its CTAs are
        // already in place then -- after this library's selection kernel, and equally after the previous layer's
        // merge when layers are issued back to back.
        cudaError_t e = rows_far ? launch_kernel(gather_update_kernel<true>, dim3((unsigned)rows), dim3(kRowThreads), 0, stream,
                                                 /*after_kernel=*/true, a)
                                 : launch_kernel(gather_update_kernel<false>, dim3((unsigned)rows), dim3(kRowThreads), 0, stream,
                                                 /*after_kernel=*/true, a);
        count_launch();
        if (e != cudaSuccess) { set_cuda_error(e); return DAF_ERR_CUDA; }
        if (int rc = check_launch()) return rc;
    }
    return DAF_OK;
}

int launch_deviation_scores(const ResolvedParams& rp, const void* k_fresh, const void* v_fresh, const void* k_cached,
                            const void* v_cached, float* scores, cudaStream_t stream) {
    if (rp.L_d == 0) return DAF_OK;
    const int warps = 8;
    int blocks = (rp.L_d + warps - 1) / warps;
    const int max_blocks = 148 * 8;          // a few waves of 256-thread CTAs; each warp then walks several tokens
    if (blocks > max_blocks) blocks = max_blocks;
    deviation_scores_kernel<<<blocks, warps * 32, 0, stream>>>(
        reinterpret_cast<const int4*>(k_fresh), reinterpret_cast<const int4*>(v_fresh),
        reinterpret_cast<const int4*>(k_cached), reinterpret_cast<const int4*>(v_cached), rp.L_d, rp.Hkv * 16, scores);
    count_launch();
    return check_launch();
}

int launch_deviation_sum(const ResolvedParams& rp, int n_sig, const void* const* k_fresh, const void* const* v_fresh,
                         const void* const* k_cached, const void* const* v_cached, float* sums, cudaStream_t stream) {
    if (rp.L_d == 0) return DAF_OK;
    if (n_sig < 1 || n_sig > kMaxSignalLayers) return DAF_ERR_INVALID_ARG;
    SignalLayers layers;
    layers.n = n_sig;
    for (int l = 0; l < kMaxSignalLayers; ++l) {
        const int j = l < n_sig ? l : 0;
        layers.k_fresh[l] = reinterpret_cast<const int4*>(k_fresh[j]);
        layers.v_fresh[l] = reinterpret_cast<const int4*>(v_fresh[j]);
        layers.k_cached[l] = reinterpret_cast<const int4*>(k_cached[j]);
        layers.v_cached[l] = reinterpret_cast<const int4*>(v_cached[j]);
    }
    const int warps = 8;
    int blocks = (rp.L_d + warps - 1) / warps;
    const int max_blocks = 148 * 8;
    if (blocks > max_blocks) blocks = max_blocks;
    deviation_sum_kernel<<<blocks, warps * 32, 0, stream>>>(layers, rp.L_d, rp.Hkv * 16, sums);
    count_launch();
    return check_launch();
}

// ------------------------------------------------ validation of caller-given positions
// The important-token stage treats "causal in packed order" as "causal by position", which holds only if the
// positions are strictly increasing; a caller who passes idx_in can have them checked on the device: each
// position must lie in [0, L_d) and exceed the one before it.  The first offence is recorded in the status
// word (DAF_ERR_BOUNDS; where = 2 out of range, 3 not increasing; detail = the offending index into idx).
__global__ void __launch_bounds__(256)
check_indices_kernel(const int32_t* __restrict__ idx, int k, int L_d, DeviceStatus* status) {
    const int i = (int)(blockIdx.x * blockDim.x + threadIdx.x);
    if (i >= k) return;
    const int p = idx[i];
    if (p < 0 || p >= L_d) report_status(status, DAF_ERR_BOUNDS, 2, i);
    else if (i > 0 && idx[i - 1] >= p) report_status(status, DAF_ERR_BOUNDS, 3, i);
}

int launch_check_indices(const int32_t* idx, int k, int L_d, DeviceStatus* status, cudaStream_t stream) {
    if (k <= 0) return DAF_OK;
    check_indices_kernel<<<(unsigned)((k + 255) / 256), 256, 0, stream>>>(idx, k, L_d, status);
    count_launch();
    return check_launch();
}

// ------------------------------------------------ offline cache stored in fp8
// Expands the document rows of an offline cache kept as 8-bit floating point (1 sign, 4 exponent, 3 mantissa
// bits, bias 7, no infinities) into the bf16 hybrid-cache buffer: element = bf16(scale[head] * value), the product in
// fp32, both roundings to nearest-even.  A streaming pass (1 byte read, 2 written per element); each thread
// takes 16 elements.
__device__ __forceinline__ float mul_rn_keep_subnormals(float a, float b) {
    float d;
    asm("mul.rn.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}
__device__ __forceinline__ uint4 expand8(uint2 bytes, float scale) {
    const __nv_fp8x2_storage_t* pr = reinterpret_cast<const __nv_fp8x2_storage_t*>(&bytes);
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __half2_raw h2 = __nv_cvt_fp8x2_to_halfraw2(pr[i], __NV_E4M3);    // exact: every value is an fp16 value
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h2));
        w[i] = pack_bf16(mul_rn_keep_subnormals(f.x, scale), mul_rn_keep_subnormals(f.y, scale));
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

__global__ void __launch_bounds__(256)
expand_fp8_cache_kernel(const uint4* __restrict__ k8, const uint4* __restrict__ v8, const float* __restrict__ k_scale,
                        const float* __restrict__ v_scale, uint4* __restrict__ kv_k, uint4* __restrict__ kv_v,
                        long long n_chunks, int Hkv) {
    pdl_launch_dependents();   // the selection kernel does not depend on this grid and may run beside it
    // chunk c = 16 consecutive elements; a head is 128 elements = 8 chunks
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x; c < 2 * n_chunks; c += stride) {
        const bool is_v = c >= n_chunks;
        const long long cc = is_v ? c - n_chunks : c;
        const int head = (int)((cc >> 3) % Hkv);
        const float* sc = is_v ? v_scale : k_scale;
        const float scale = sc != nullptr ? __ldg(sc + head) : 1.0f;
        const uint4 in = __ldcs((is_v ? v8 : k8) + cc);
        uint4* out = (is_v ? kv_v : kv_k) + 2 * cc;
        out[0] = expand8(make_uint2(in.x, in.y), scale);
        out[1] = expand8(make_uint2(in.z, in.w), scale);
    }
}

int launch_expand_fp8(const ResolvedParams& rp, const void* k8, const void* v8, const float* k_scale, const float* v_scale,
                      void* kv_k, void* kv_v, cudaStream_t stream) {
    const long long n_chunks = (long long)rp.L_d * rp.Hkv * 8;     // 16-element chunks per tensor
    if (n_chunks == 0) return DAF_OK;
    long long blocks = (2 * n_chunks + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    expand_fp8_cache_kernel<<<(unsigned)blocks, 256, 0, stream>>>(
        reinterpret_cast<const uint4*>(k8), reinterpret_cast<const uint4*>(v8), k_scale, v_scale,
        reinterpret_cast<uint4*>(kv_k), reinterpret_cast<uint4*>(kv_v), n_chunks, rp.Hkv);
    count_launch();
    return check_launch();
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
    fuse_rows_kernel<<<rows, kRowThreads, 0, stream>>>(a);
    count_launch();
    return check_launch();
}

}  // namespace daf
