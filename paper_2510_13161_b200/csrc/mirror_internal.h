// Internal definitions shared by the library's translation units (never installed).
#pragma once
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mirror.h"

// ----------------------------------------------------------------------------------------------
// context
// ----------------------------------------------------------------------------------------------
struct MirrorTreeInfo {            // host-side digest of one token tree, rebuilt per call (cheap)
    int n = 0, n_branches = 0, max_len = 0;
    unsigned long long anc[MIRROR_MAX_NODES][2];   // bit j of anc[i]: node j is i or an ancestor of i
    int parent[MIRROR_MAX_NODES];
    int depth[MIRROR_MAX_NODES];
    unsigned char path[MIRROR_MAX_BRANCHES][MIRROR_MAX_DEPTH];   // node ids along each branch (below the root)
    unsigned char path_len[MIRROR_MAX_BRANCHES];
};

// Tuning values, read ONCE from the environment when a context is created (defaults measured on B200); a context made
// on the stack by the no-allocation entry point keeps the defaults.  The last two exist for the tests of the bounded
// waits: a short limit, and a producer that stops issuing copies after a number of stages, so that a consumer's wait
// runs out and the kernel has to unwind (nothing traps, nothing spins without limit, no memory fault is provoked).
struct MirrorTuning {
    int attn_groups = 0;             // MIRROR_ATTN_GROUPS: upper limit of CTA groups (0: all)
    int attn_whole_units = 1;        // MIRROR_ATTN_WHOLE_UNITS: 0 = never trade CTA groups for whole units
    int attn_snap = 4;               // MIRROR_ATTN_SNAP: boundary snapping distance in tiles
    int attn_ring = 0;               // MIRROR_ATTN_RING: K/V ring depths as two digits, e.g. 64 (0: deepest that fits)
    int lm_pair2_max_rows = 128;     // MIRROR_LM_PAIR2_MAX_ROWS: two CTAs per SM up to this many rows
    int lm_ctas_per_sm = 0;          // MIRROR_LM_CTAS_PER_SM: 1 or 2 (0: by rows)
    int lm_stages = 0;               // MIRROR_LM_STAGES: fewer pipeline stages than fit (0: all)
    int lm_rows = 0;                 // MIRROR_LM_ROWS: rows per CTA and unit of the LM head as a weight stream (0: balanced choice)
    int lm_pair_min_rows = 1;        // MIRROR_LM_PAIR_MIN_ROWS: rows from which the pair kernel is used
    int lm_kgroup = 0;               // MIRROR_LM_KGROUP: K blocks requested at a time by the single-CTA kernel (0: default)
    long long wait_limit_cycles = 4000000000ll;   // MIRROR_WAIT_LIMIT_CYCLES: SM cycles after which a device-side wait gives up
    int test_stall_after = -1;       // MIRROR_TEST_STALL_AFTER_STAGES: a producer issues this many stages, then stops (-1: off);
                                     // applies to the FIRST attention launch and the first LM-head launch of a context only
    int test_stall_attn_left = 1, test_stall_lm_left = 1;
};
void mirror_tuning_from_env(MirrorTuning* t);

// mirror_verify_step_host copies and attends to a step's layers in this many pieces (the last layer first, alone).  The
// pieces' copies are what bounds the host-buffer step on a large model (1.7 GB of Q per step on the 66B-class workload),
// and the last piece's attention is what is left exposed behind them, so the pieces are kept small.
constexpr int kMirrorHostChunks = 12;
struct mirror_ctx {
    mirror_model_desc desc;
    MirrorTuning tune;
    int device = 0;
    int num_sms = 0;
    float scale = 0.f;
    float temperature = 1.f;
    int* d_status = nullptr;        // [2]: {code, detail}
    void* ws = nullptr;
    size_t ws_bytes = 0;
    long long launches = 0;
    bool lm_attr_set = false;
    bool lm_pair_attr_set = false;
    cudaEvent_t stage_ev[4] = {nullptr, nullptr, nullptr, nullptr};
    bool stage_ev_on = false;
    cudaStream_t copy_stream = nullptr;                     // mirror_verify_step_host: created on first use
    cudaEvent_t copy_ev[kMirrorHostChunks + 1] = {};
    PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
};

mirror_status mirror_build_tree(const mirror_tree* tree, MirrorTreeInfo* info);

// Workspace carving.  The layout depends only on the model shape and the row count M, so every entry
// point finds the same regions: [zeroed words | attention split records | LM-head partials | lse, argmax
// scratch | fp32 logits | fp64 acceptance scratch].  Offsets are 256-byte aligned; the first region is zeroed when the workspace is attached.
constexpr size_t kWsZeroedBytes = 4096;     // words at the front of the workspace that are zero between launches (none in use now)
struct MirrorWsLayout {
    size_t zeroed = 0;                                   // kWsZeroedBytes of zeroed words
    size_t attn_partial = 0, attn_partial_bytes = 0;     // split-KV partial accumulators
    size_t lm_partial = 0, lm_partial_bytes = 0;         // per-CTA (or per-unit) row partials
    size_t lse = 0, argmax = 0;                          // [M] scratch each
    size_t logits = 0, logits_bytes = 0;                 // fp32 [M, V]
    size_t accept_scratch = 0;                           // fp64 [B, 2, V]: running distribution of the tree acceptance
    size_t lm_topk = 0, lm_topk_bytes = 0;               // per partial and row: the MIRROR_MAX_TOPK best (logit, id) pairs of the fused Top-kappa
    size_t end_attn = 0, end_lmhead = 0, end_logits = 0, end_accept = 0, end_topk = 0;   // bytes needed up to each region
};
void mirror_ws_layout(const mirror_ctx* ctx, size_t M, MirrorWsLayout* out, size_t B = 0);

mirror_status mirror_accept_launch(mirror_ctx* ctx, const mirror_tree* tree, const MirrorTreeInfo& ti,
                                   const mirror_accept_in* in, const mirror_accept_out* out, cudaStream_t stream,
                                   double* tree_scratch = nullptr);
mirror_status mirror_lmhead_launch(mirror_ctx* ctx, const void* hidden, int M, const void* W, int topk,
                                   const int32_t* gather_row, const int32_t* gather_tok, int n_gather,
                                   int32_t* argmax, float* maxlogit, float* lse, int32_t* topk_id,
                                   float* topk_logprob, float* gather_logit, float* logits_out,
                                   void* partial_ws, size_t partial_bytes, float* lse_scratch, cudaStream_t stream,
                                   cudaEvent_t after_gemm = nullptr, void* topk_logprob_bf16 = nullptr,
                                   void* topk_ws = nullptr, size_t topk_ws_bytes = 0);
// LM-head GEMM + per-unit row partials on CTA pairs (many hidden rows); *n_partials partials of [M] rows are left in
// partial_ws for lmhead_merge_kernel.  mirror_lmhead_pair_partials(V) is that count.
int mirror_lmhead_pair_partials(int V);
// Can the Top-kappa of M rows be selected inside the GEMM's epilogue?  (One row chunk, and four lists per CTA and row in
// shared memory beside a pipeline that is still deep enough.)
bool mirror_lmhead_topk_fusable(const mirror_ctx* ctx, int M, int topk);
// w_scale / h_scale non-null: W and hidden are e4m3 bytes with one scale per row (the GEMM runs on kind::f8f6f4).
mirror_status mirror_lmhead_pair_launch(mirror_ctx* ctx, const void* hidden, int M, const void* W, float* logits_out,
                                        void* partial_ws, size_t partial_bytes, cudaStream_t stream, int* n_partials,
                                        const float* w_scale = nullptr, const float* h_scale = nullptr,
                                        int topk = 0, void* topk_ws = nullptr, size_t topk_ws_bytes = 0);
// Plain GEMM on CTA pairs: partial[s][M][N] (fp32) = x[M, K-slice s] * W[N, K-slice s]^T for the *k_slices slices that
// mirror_linear_slices() picks (1 when the output tiles alone fill the GPU); the caller adds the slices in order.
int mirror_linear_slices(const mirror_ctx* ctx, int M, int N, int K);
mirror_status mirror_linear_partial_launch(mirror_ctx* ctx, const void* x, int M, const void* W, int N, int K, float* partial,
                                           size_t partial_bytes, cudaStream_t stream, int* k_slices);
// e4m3 cache for mirror_attn_launch: pools, k_new and v_new hold codes; device scales per (layer, KV head), host Q scale.
struct MirrorAttnFp8 {
    const float* k_scale;
    const float* v_scale;
    float q_scale;
};
// e4m3 codes of a bf16 K or V tensor under given scales (see mirror_kv_quantize_fp8), launched with programmatic stream
// serialization.
mirror_status mirror_kv_quantize_launch(mirror_ctx* ctx, const void* x, int n_layers, int64_t layer_stride, int64_t layer_elems,
                                       int inner, const float* scale, void* out_fp8, cudaStream_t stream);
mirror_status mirror_attn_launch(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const MirrorTreeInfo& ti,
                                 const void* q, const void* k_new, const void* v_new, void* out, float* lse_out,
                                 float* partial_ws, cudaStream_t stream, const MirrorAttnFp8* f8 = nullptr);

// bf16 tensor map with 128-byte swizzle.  dims/box are innermost-first; strides_bytes[i] is the byte
// stride of dimension i+1 (rank-1 entries).
mirror_status mirror_make_tmap(const mirror_ctx* ctx, CUtensorMap* map, const void* base, int rank,
                               const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box);

#define MIRROR_CUDA_OK(expr)                          \
    do {                                              \
        cudaError_t e__ = (expr);                     \
        if (e__ != cudaSuccess) return MIRROR_ERR_CUDA; \
    } while (0)

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// device status codes written into d_status[0]
#define MIRROR_DEV_TIMEOUT 7
#define MIRROR_DEV_CHECK 6

#ifdef __CUDACC__
// ----------------------------------------------------------------------------------------------
// PTX wrappers (sm_100a)
// ----------------------------------------------------------------------------------------------
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

#ifndef MIRROR_PARK_NS
#define MIRROR_PARK_NS 20000u
#endif
// try_wait that lets the hardware park the thread (up to `ns` nanoseconds) until the phase completes, instead of
// returning at once: a hot spin on try_wait issues a shared-memory operation every few cycles and starves the
// warps that share the SM's shared-memory pipeline.
__device__ __forceinline__ bool mbar_try_wait_park(uint64_t* bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}

// Bounded wait.  One plain try_wait first (the common case: the phase is already complete); after that the
// thread parks in the barrier unit for up to 20 us at a time and keeps an eye on the SM cycle counter: it gives
// up after `limit_cycles` (about 2 s at 2 GHz by default).  Returns false on expiry; the caller then records
// the failure and unwinds (no trap, no endless spin).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, long long limit_cycles = 4000000000ll) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait_park(bar, parity, MIRROR_PARK_NS)) return true;
        if (clock64() - t0 > limit_cycles) return false;
    }
}

// ---- TMA -------------------------------------------------------------------------------------
__device__ __forceinline__ void prefetch_tmap(const void* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const void* map, uint64_t* bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d_hint(void* smem_dst, const void* map, uint64_t* bar, int x, int y,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_load_5d(void* smem_dst, const void* map, uint64_t* bar, int c0, int c1, int c2,
                                            int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_normal() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// ---- tcgen05 / TMEM --------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {   // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {         // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem desc] * B[smem desc], bf16 inputs, fp32 accumulate; one thread issues.
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Same, with the two 64-bit descriptors passed as 32-bit halves (the issuing thread keeps the constant halves in
// registers and only adds to the low words: it is a single thread on the critical path).
__device__ __forceinline__ void umma_f16_lohi(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                              uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
// A operand read from tensor memory (row i of A in TMEM lane i, two 16-bit elements per 32-bit column),
// B from a shared-memory descriptor.
__device__ __forceinline__ void umma_f16_tmem_a(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                                uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
// low / high words of a 128-byte-swizzle shared-memory descriptor
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t addr, uint32_t lbo_bytes) {
    return ((addr & 0x3FFFF) >> 4) | ((lbo_bytes >> 4) << 16);
}
__device__ __forceinline__ uint32_t umma_desc_hi_sw128(uint32_t sbo_bytes) {
    return (sbo_bytes >> 4) | (1u << 14) | (2u << 29);
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Arrive on an mbarrier once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread t of the warp reads lane (base_lane + t).
__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t (&r)[32]) {
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
__device__ __forceinline__ void tmem_ld_32x32b_x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 64 bf16 (128 B),
// 8-row groups 1024 B apart.  `addr` is the shared-window byte address of the (sub)tile.
__device__ __forceinline__ uint64_t umma_desc_k_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);          // start address
    d |= (uint64_t)1 << 16;                          // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                          // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                          // 128-byte swizzle
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, tile M x N.
__host__ __device__ __forceinline__ uint32_t umma_idesc_bf16(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Programmatic dependent launch: a kernel launched with mirror_launch_pdl may be scheduled while the kernel before it
// in the stream is still running; grid_dep_wait() blocks until that kernel has completed and its memory is visible
// (a no-op for a plain launch), grid_dep_launch() lets the kernel after this one be scheduled as SMs free up.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

}  // namespace ptx

template <typename... KArgs, typename... Args>
inline cudaError_t mirror_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif  // __CUDACC__
