// Shared host/device helpers of the DAF library: status codes, launch
// accounting, and thin wrappers around the sm_100a PTX this library issues
// (mbarrier, TMA, tcgen05).  Everything here is internal to the CUDA path.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/daf.h"

namespace daf {

// ---------------------------------------------------------------- host side
void set_cuda_error(cudaError_t e);
void count_launch(int n = 1);
int check_launch();  // cudaGetLastError -> DAF_OK / DAF_ERR_CUDA

// The status word lives in the first bytes of the caller's workspace.
constexpr size_t kStatusBytes = 256;
struct DeviceStatus {
    int code;      // 0, or DAF_ERR_TIMEOUT / DAF_ERR_BOUNDS
    int where;     // a small tag naming the wait or index that failed
    int block;     // linear block id that reported first
    int detail;
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct ResolvedParams {
    int L_d, L_q, N, Hq, Hkv, G, k;
    float scale;
    int fuse_mode, overwrite;
};
int resolve_params(const daf_params* p, ResolvedParams* out);  // validates; DAF_OK or error

// kernel launchers (daf_select.cu, daf_attn.cu), called by the C ABI in daf_api.cu
size_t select_scratch_bytes(int L_d);
int launch_select(const ResolvedParams& rp, const float* scores, int n_sig, const int32_t* idx_in,
                  const void* q_fresh, const void* k_fresh, const void* v_fresh, void* kv_k, void* kv_v,
                  int32_t* idx_out, void* q_pack, void* k_pack, void* v_pack,
                  DeviceStatus* status, void* scratch, cudaStream_t stream, bool scores_from_previous_kernel = false,
                  bool beside_previous_kernel = false, bool select_only = false, bool rows_far = false);
int launch_check_indices(const int32_t* idx, int k, int L_d, DeviceStatus* status, cudaStream_t stream);
int launch_expand_fp8(const ResolvedParams& rp, const void* k8, const void* v8, const float* k_scale, const float* v_scale,
                      void* kv_k, void* kv_v, cudaStream_t stream);
constexpr int kMaxSignalLayersHost = 8;
int launch_deviation_sum(const ResolvedParams& rp, int n_sig, const void* const* k_fresh, const void* const* v_fresh,
                         const void* const* k_cached, const void* const* v_cached, float* sums, cudaStream_t stream);
int launch_fuse(const ResolvedParams& rp, const int32_t* idx, const void* o_imp, const void* o_q, void* hidden,
                int32_t* row_pos_out, cudaStream_t stream);
int launch_deviation_scores(const ResolvedParams& rp, const void* k_fresh, const void* v_fresh, const void* k_cached,
                            const void* v_cached, float* scores, cudaStream_t stream);
struct AttnPlan { int Gp, Tt, n_tb, head_blocks, n_splits, tiles_per_split; };
AttnPlan plan_attention(int n_q, int n_kv, int Hq, int G, int causal_off, bool pack_group, bool allow_split);
size_t attn_partial_bytes(int n_q, int Hq, int n_splits);
int launch_attention(const void* q, const void* k, const void* v, int n_q, int n_kv, int Hq, int Hkv, int causal_off,
                     float scale, bool pack_group, bool allow_split, void* out, long long out_row_stride_bytes,
                     const int32_t* dst_rows, float* lse, DeviceStatus* status, void* scratch, size_t scratch_bytes,
                     cudaStream_t stream, bool after_kernel = false, const int32_t* q_pos = nullptr);
// Steps 2 and 3 of a layer from one list of work items (one attention launch and one merge launch).
struct JointPlan {
    int n_tb_i, chunk, n_slots, items_i;                                  // important-token stage
    int Gp_q, Tt_q, n_tb_q, head_blocks_q, n_splits_q, tiles_per_split_q, items_q;   // question stage
    size_t part_bytes_q, part_bytes_i;        // partial results of each stage
};
JointPlan plan_joint(int k, int L_q, int L_d, int Hq, int G);
size_t joint_partial_bytes(const JointPlan& jp);
int launch_bounded_wait_selftest(DeviceStatus* status, int limit_ms, cudaStream_t stream);
// q_imp == nullptr: the important rows' Q is read in place, row idx[j] of q_fresh;
// k_imp == nullptr (then v_imp too): their K and V are read in place, rows idx[j] of k_fresh / v_fresh
int launch_attention_joint(const void* q_imp, const void* q_fresh, const int32_t* idx, const void* k_imp, const void* v_imp,
                           const void* k_fresh, const void* v_fresh,
                           int k, void* out_imp, const int32_t* dst_rows_imp, const void* q_question, const void* kv_k,
                           const void* kv_v,
                           int L_q, int L_d, void* out_question, long long out_row_stride_bytes, int Hq, int Hkv,
                           float scale, DeviceStatus* status, void* scratch, size_t scratch_bytes, cudaStream_t stream,
                           bool after_kernel, int launches = 3);   // launches: bit 0 the attention launch, bit 1 the merge

// ---------------------------------------------------------------- device side
#ifdef __CUDACC__

// Launch helper.  With `after_kernel` the launch carries the programmatic-serialization attribute:
// the kernel may start while the previous kernel of the stream is still draining and must call
// pdl_wait() before it touches anything that kernel wrote.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 bool after_kernel, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = after_kernel ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Programmatic dependent launch: wait for the preceding kernel's results / let the next kernel start launching.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void report_status(DeviceStatus* st, int code, int where, int detail) {
    if (st != nullptr && atomicCAS(&st->code, 0, code) == 0) {
        st->where = where;
        st->block = (int)(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z));
        st->detail = detail;
    }
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// True in exactly one lane of a converged warp (the same lane every time).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
// Bounded wait: gives up after `limit` polls or as soon as another thread of the
// CTA has raised *abort_flag.  Returns false on give-up (the caller unwinds).
constexpr uint32_t kWaitLimitPolls = 1u << 22;          // hard cap on polls
constexpr unsigned long long kWaitLimitNs = 1000000000ull;  // and one second of wall time
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#ifdef DAF_TRACE
// Debug build only (-DDAF_TRACE): first-start / last-end time of each kernel, one table per source file.
#define DAF_KT_TABLE static __device__ unsigned long long g_kt[32]
#define DAF_KT_BEGIN(id) do { if (threadIdx.x == 0) atomicMin(&g_kt[2 * (id)], global_ns()); } while (0)
#define DAF_KT_END(id) do { if (threadIdx.x == 0) atomicMax(&g_kt[2 * (id) + 1], global_ns()); } while (0)
#define DAF_KT_READER(name)                                                                   \
    extern "C" int name(void* host, int reset) {                                              \
        if (reset) {                                                                          \
            unsigned long long init[32];                                                      \
            for (int i = 0; i < 32; ++i) init[i] = (i & 1) ? 0ull : ~0ull;                    \
            return (int)cudaMemcpyToSymbol(g_kt, init, sizeof(init));                         \
        }                                                                                     \
        return (int)cudaMemcpyFromSymbol(host, g_kt, 32 * sizeof(unsigned long long));        \
    }
#else
#define DAF_KT_BEGIN(id) do {} while (0)
#define DAF_KT_END(id) do {} while (0)
#endif
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          DeviceStatus* st, int where, unsigned long long limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t it = 0; it < kWaitLimitPolls; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 31u) == 31u) {
            if (*abort_flag != 0) return false;
            if (global_ns() - t0 > limit_ns) break;
        }
    }
    *abort_flag = 1;
    report_status(st, DAF_ERR_TIMEOUT, where, (int)parity);
    return false;
}

// ---- TMA (tiled bulk tensor loads into shared memory, completion on an mbarrier)
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// Tiled store of a shared-memory tile to global memory (bulk-group completion).
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* m, const void* src, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// waits until the bulk stores committed so far have finished reading shared memory
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// ---- cp.async (16-byte copies global -> shared by ordinary threads; used where rows are fetched through an index)
// copies 16 bytes, or writes 16 zero bytes when src_bytes == 0 (src must still be a valid address)
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// makes this thread's earlier shared-memory writes visible to the asynchronous proxy (TMA, tensor cores)
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- tcgen05 (5th-generation tensor cores, accumulators in tensor memory)
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Arrive on an mbarrier once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp gets lane (base lane + t).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}

// Shared-memory matrix descriptor for tcgen05.mma operands stored in the
// 128-byte-swizzled layout TMA writes (rows of 128 bytes, 8-row groups of 1024
// bytes).  lbo/sbo are the leading/stride byte offsets of the canonical layout.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of this architecture
    d |= (uint64_t)2 << 61;  // 128-byte swizzle
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, M x N tile, A K-major, B K-major or MN-major.
__host__ __device__ constexpr uint32_t make_idesc_bf16(uint32_t M, uint32_t N, uint32_t b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major << 16) | ((N >> 3) << 17) | ((M >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Two-wide fp32 arithmetic (one instruction for a pair of floats held in a 64-bit register)
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ float f32x2_lo(uint64_t v) {
    [[maybe_unused]] float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    (void)hi;
    return lo;
}
__device__ __forceinline__ float f32x2_hi(uint64_t v) {
    [[maybe_unused]] float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    (void)lo;
    return hi;
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fmul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

#endif  // __CUDACC__
}  // namespace daf
