// LM head for many hidden rows (Eq. 1 over the B * (1 + kappa*gamma) rows of a batched verify step): the same fused
// GEMM + row reductions as lmhead_kernel, issued on CTA PAIRS (tcgen05 cta_group::2).
//
// Why a second kernel: with M >= ~200 rows the LM head stops being a weight stream and becomes a GEMM, and a
// single-CTA 128 x N tile asks the L2 for more bytes per flop than it delivers.  A pair of CTAs (the two SMs of a
// TPC) runs one UMMA of 256 vocabulary rows x N hidden rows per K step: each CTA stages its own 128 weight rows and
// only HALF of the hidden rows, and the tensor cores of both SMs read both halves.  Per K block of 64 a CTA loads
// 16 KB + N/2 * 128 B for 128 * N * 64 * 2 flop: 131 flop/B at N = 256 against 79 flop/B before.
//
// Work unit = (256-row vocabulary tile, row chunk of N <= 256 hidden rows).  Units are dealt to the pairs round-robin
// in the order (tile major, chunk minor), so that at any time the pairs work on a handful of neighbouring tiles and
// the chunks of one tile run on different pairs at the same moment: every weight tile leaves HBM once and the other
// chunks hit it in L2.  Each unit leaves one partial (max, argmax, sum-exp) per hidden row and 128-row half tile;
// lmhead_merge_kernel folds them in a fixed order, so the result does not depend on which pair ran which unit.
//
// Per CTA, 6 warps as in lmhead_kernel: warp 0 TMA producer (own W rows + own half of the hidden chunk), warp 1
// TMEM owner; in the pair's leader (cluster rank 0) its elected lane issues the UMMAs for both CTAs; warps 2..5
// epilogue over the CTA's own 128 accumulator lanes.
// Barriers that the other CTA signals: the copies of BOTH CTAs complete their bytes on the leader's `full` barrier
// (the peer's TMA names the leader's barrier; no thread sits in between), the UMMA completion is committed with a
// multicast arrive to `empty` / `acc_full` of both CTAs, and the peer's epilogue warps arrive remotely on the leader's
// `acc_empty`.  Every wait is bounded; both CTAs meet at a cluster barrier before the TMEM is released.
#include <math.h>
#include <stdlib.h>

#include "mirror_internal.h"

namespace {

constexpr int kThreads = 192;
constexpr int kBK = 64;
constexpr int kTileV = 128;                 // vocabulary rows per CTA and unit
constexpr int kPairV = 2 * kTileV;          // per pair
constexpr int kATileBytes = kTileV * kBK * 2;
constexpr int kMaxStages = 8;
constexpr int kAcc = 2;
constexpr int kMaxChunkRows = 256;
constexpr int kSmemBudget = 232448;
constexpr int kCtrlBytes = 1024 + 4 * kMaxChunkRows * 12;

struct PairParams {
    int M, V, H;
    int n_chunks, chunk_rows, half_rows;
    int acc_stride, tmem_cols;
    int stages, stage_bytes;
    int rows_cta, a_bytes;                  // vocabulary rows a CTA loads per unit (<= 128, a multiple of 8) and their bytes per stage
    int ctas_per_sm;                        // 2 when few rows leave room for two CTAs' pipelines on an SM
    int k_slices, kb_per_slice;             // split-K (plain GEMM mode only): K blocks of 64 per unit
    int n_units;
    int w_keep;                             // 1: weight tiles are re-read by other chunks, keep them in L2
    float inv_T, inv_T_log2e;
    float* logits_out;                      // reduce mode: nullable [M, V]; plain GEMM mode: [k_slices][M, V] partial sums
    float* part_max;                        // [partials][M]
    int* part_idx;
    float* part_sum;
    int* status;
    int topk;                               // > 0: the epilogue keeps each row's topk best (logit, id) pairs per CTA or unit
    int topk_bytes;                         // shared memory of those lists
    float* part_topv;                       // [partials][M][topk]
    int* part_topi;
    int fp8;                                // 1: W and the hidden rows are e4m3 bytes (K counted in 128-byte blocks all the same)
    const float* w_scale;                   // fp8: [V] scale of each weight row
    const float* h_scale;                   // fp8: [M] scale of each hidden row
    long long wait_limit;                   // SM cycles after which a wait gives up
    int stall_after;                        // test aid: the producers stop after this many stages (-1: never)
};

struct Ctrl {
    uint64_t full[kMaxStages];              // leader only: the stage has landed in both CTAs (transaction bytes of both)
    uint64_t empty[kMaxStages];             // UMMAs that read the stage have completed (multicast commit)
    uint64_t acc_full[kAcc];                // accumulator complete (multicast commit)
    uint64_t acc_empty[kAcc];               // leader only: 4 + 4 epilogue warps have drained the accumulator
    uint32_t tmem_base;
    volatile int abort;
};

__device__ __forceinline__ void fail(const PairParams& p, Ctrl* c, int where) {
    c->abort = 1;
    if (atomicCAS(p.status, 0, MIRROR_DEV_TIMEOUT) == 0) atomicExch(p.status + 1, where);
}

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {      // every thread of both CTAs
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory object in the CTA of rank `rank`
__device__ __forceinline__ uint32_t map_to_rank(const void* smem_ptr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(ptx::smem_u32(smem_ptr)), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// bounded wait on a barrier that the other CTA of the pair arrives on
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, long long limit_cycles = 4000000000ll) {
    const uint32_t a = ptx::smem_u32(bar);
    const long long t0 = clock64();
    for (;;) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(a), "r"(parity), "r"(MIRROR_PARK_NS)
            : "memory");
        if (ok) return true;
        if (clock64() - t0 > limit_cycles) return false;
    }
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t ncols) {    // one warp of EACH CTA
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ptx::smem_u32(smem_result)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {         // one warp of EACH CTA
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// TMA load into this CTA's shared memory whose bytes are counted on a barrier of the pair's leader (cluster address)
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const void* map, uint32_t bar_cluster_addr, int x, int y,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(ptx::smem_u32(smem_dst)), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y), "l"(policy)
        : "memory");
}
// D[tmem of both CTAs] (+)= A (128 rows from each CTA's shared memory) * B (N/2 rows from each CTA's shared memory)
__device__ __forceinline__ void umma_pair_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                              uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// the same for e4m3 operands (32 elements of K per instruction: the same 32 bytes of a 128-byte swizzled row)
__device__ __forceinline__ void umma_pair_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// instruction descriptor for e4m3 x e4m3 -> fp32, both operands K-major
__host__ __device__ __forceinline__ uint32_t umma_idesc_e4m3(int M, int N) {
    return (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// arrive on the barrier at this shared-memory offset in BOTH CTAs once all UMMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(ptx::smem_u32(bar)), "h"((uint16_t)3)
                 : "memory");
}

// Fused Top-kappa (Eq. 6).  Every epilogue warp keeps, for every hidden row, its own sorted list of K (logit, id) pairs in
// shared memory (order: logit descending, id ascending); lane j owns the lists of the rows in column j of each 32-column
// group, so 32 rows are updated side by side and nothing is locked.  A list lives as long as the CTA (one row chunk: the CTA
// meets the same rows in every unit), so after the first tiles only a few logits pass its last entry.
__device__ __forceinline__ void topk_list_insert(float* lv, int* li, int K, float x, int xi) {
    int i = K - 1;
    if (!(x > lv[i] || (x == lv[i] && xi < li[i]))) return;
    while (i > 0 && (x > lv[i - 1] || (x == lv[i - 1] && xi < li[i - 1]))) { lv[i] = lv[i - 1]; li[i] = li[i - 1]; --i; }
    lv[i] = x;
    li[i] = xi;
}

// kReduce: LM head (row reductions in the epilogue, optional spill).  !kReduce: plain GEMM C = W h^T for the layer
// projections, split along K when there are fewer tiles than CTA pairs; the epilogue only stores fp32 partial sums.
// kFp8 / kTopk: e4m3 operands with per-row scales / Top-kappa lists in the epilogue, as separate instantiations so that
// the plain bf16 head carries none of their registers and branches.
template <bool kReduce, bool kFp8, bool kTopk>
__device__ __forceinline__ void pair_gemm_body(const CUtensorMap& tm_w, const CUtensorMap& tm_h, const PairParams& p) {
    extern __shared__ uint8_t smem_raw[];
    // (the dynamic shared window starts at the same offset in both CTAs, so the aligned layout is the same too)
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_base = smem;
    Ctrl* ctrl = (Ctrl*)(smem + (size_t)p.stages * p.stage_bytes);
    float* st_max = (float*)((uint8_t*)ctrl + 1024);          // [4][kMaxChunkRows]
    int* st_idx = (int*)(st_max + 4 * kMaxChunkRows);
    float* st_sum = (float*)(st_idx + 4 * kMaxChunkRows);
    float* tk_val = (float*)((uint8_t*)ctrl + kCtrlBytes);    // [4 warps][chunk_rows][topk]  (only when p.topk > 0)
    int* tk_idx = (int*)(tk_val + (size_t)4 * p.chunk_rows * p.topk);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_rank();
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int n_kb = p.H / kBK;
    // unit -> (vocabulary tile, K slice, row chunk); chunk fastest, so the chunks of a tile run side by side
    auto decode = [&](int u, int& tile, int& slice, int& chunk) {
        chunk = u % p.n_chunks;
        const int t2 = u / p.n_chunks;
        slice = t2 % p.k_slices;
        tile = t2 / p.k_slices;
    };

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(&ctrl->full[s], 1);
            ptx::mbar_init(&ctrl->empty[s], 1);
        }
        for (int a = 0; a < kAcc; ++a) { ptx::mbar_init(&ctrl->acc_full[a], 1); ptx::mbar_init(&ctrl->acc_empty[a], 8); }
        ctrl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tm_w);
        ptx::prefetch_tmap(&tm_h);
    }
    if (warp == 1) {
        tmem_alloc_pair(&ctrl->tmem_base, (uint32_t)p.tmem_cols);
        tmem_relinquish_pair();
    }
    ptx::tc_fence_before();
    __syncthreads();
    cluster_sync_all();                 // the other CTA's barriers exist before anything arrives on them
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            const uint64_t pol_w = p.w_keep ? ptx::policy_evict_normal() : ptx::policy_evict_first();
            const uint64_t pol_h = ptx::policy_evict_last();
            int s = 0, n_issued = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int u = pair; u < p.n_units && ok; u += n_pairs) {
                int tile, slice, chunk;
                decode(u, tile, slice, chunk);
                const int w_row = (tile * 2 + (int)rank) * p.rows_cta;
                const int h_row = chunk * p.chunk_rows + (int)rank * p.half_rows;
                const int kb_end = min(n_kb, (slice + 1) * p.kb_per_slice);
                for (int kb = slice * p.kb_per_slice; kb < kb_end; ++kb) {
                    if (p.stall_after >= 0 && n_issued >= p.stall_after) { ok = false; break; }       // (test aid: neither arms nor copies)
                    if (ctrl->abort || !ptx::mbar_wait(&ctrl->empty[s], ph ^ 1, p.wait_limit)) { fail(p, ctrl, 11); ok = false; break; }
                    if (rank == 0) ptx::mbar_arrive_expect_tx(&ctrl->full[s], 2u * (uint32_t)p.stage_bytes);
                    const uint32_t bar = map_to_rank(&ctrl->full[s], 0);
                    uint8_t* dst = stage_base + s * p.stage_bytes;
                    tma_load_2d_pair(dst, &tm_w, bar, kb * kBK, w_row, pol_w);
                    tma_load_2d_pair(dst + p.a_bytes, &tm_h, bar, kb * kBK, h_row, pol_h);
                    ++n_issued;
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                }
            }
            // (copies still in flight after a failure: the leader's issuer or its 2 s limit outlasts them, and both CTAs
            // meet at the cluster barrier below before either one's shared memory goes away)
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // -------------------------------------------------------------- UMMA issuer (leader)
            const uint32_t idesc = kFp8 ? umma_idesc_e4m3(kPairV, p.chunk_rows) : ptx::umma_idesc_bf16(kPairV, p.chunk_rows);
            const uint32_t stage_u32 = ptx::smem_u32(stage_base);
            int s = 0, ab = 0;
            uint32_t ph = 0, aph = 0;
            bool ok = true;
            for (int u = pair; u < p.n_units && ok; u += n_pairs) {
                if (ctrl->abort || !mbar_wait_cluster(&ctrl->acc_empty[ab], aph ^ 1, p.wait_limit)) { fail(p, ctrl, 12); ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(ab * p.acc_stride);
                int tile, slice, chunk;
                decode(u, tile, slice, chunk);
                const int nk = min(n_kb, (slice + 1) * p.kb_per_slice) - slice * p.kb_per_slice;
                for (int kb = 0; kb < nk; ++kb) {
                    if (ctrl->abort || !ptx::mbar_wait(&ctrl->full[s], ph, p.wait_limit)) { fail(p, ctrl, 13); ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t sa = stage_u32 + (uint32_t)(s * p.stage_bytes);
                    const uint32_t sb = sa + (uint32_t)p.a_bytes;
                    if constexpr (kFp8) {
#pragma unroll
                        for (int k4 = 0; k4 < kBK / 16; ++k4)
                            umma_pair_f8(d_tmem, ptx::umma_desc_k_sw128(sa + k4 * 32), ptx::umma_desc_k_sw128(sb + k4 * 32), idesc,
                                         (kb | k4) != 0);
                    } else {
#pragma unroll
                        for (int k4 = 0; k4 < kBK / 16; ++k4)
                            umma_pair_f16(d_tmem, ptx::umma_desc_k_sw128(sa + k4 * 32), ptx::umma_desc_k_sw128(sb + k4 * 32), idesc,
                                          (kb | k4) != 0);
                    }
                    umma_commit_pair(&ctrl->empty[s]);
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                }
                if (ok) umma_commit_pair(&ctrl->acc_full[ab]);
                if (++ab == kAcc) { ab = 0; aph ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs, own 128 lanes)
        const int q = warp & 3;
        float* my_max = st_max + q * kMaxChunkRows;
        int* my_idx = st_idx + q * kMaxChunkRows;
        float* my_sum = st_sum + q * kMaxChunkRows;
        const int n_cg = (p.chunk_rows + 31) / 32;
        // the four warps hold disjoint vocabulary rows: one partial per hidden row out of their four states
        auto flush = [&](size_t pbase, int rbase) {
            for (int c = (warp - 2) * 32 + lane; c < p.chunk_rows; c += 128) {
                const int row = rbase + c;
                if (row >= p.M) continue;
                float m = -INFINITY, s = 0.f;
                int idx = 0x7fffffff;
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const float pm = st_max[w * kMaxChunkRows + c], ps = st_sum[w * kMaxChunkRows + c];
                    const int pi = st_idx[w * kMaxChunkRows + c];
                    if (pm == -INFINITY) continue;
                    if (pm > m || (pm == m && pi < idx)) {
                        s = ps + (m == -INFINITY ? 0.f : s * exp2f((m - pm) * p.inv_T_log2e));
                        m = pm; idx = pi;
                    } else {
                        s += ps * exp2f((pm - m) * p.inv_T_log2e);
                    }
                }
                p.part_max[pbase + row] = m;
                p.part_idx[pbase + row] = idx;
                p.part_sum[pbase + row] = s;
                // each warp's list is a partial list of its own: [4 * CTA + warp][row][topk]
                for (int w = 0; w < 4 && kTopk; ++w)
                    for (int i = 0; i < p.topk; ++i) {
                        const size_t at = (((size_t)blockIdx.x * 4 + w) * p.M + row) * p.topk + i;
                        p.part_topv[at] = tk_val[((size_t)w * p.chunk_rows + c) * p.topk + i];
                        p.part_topi[at] = tk_idx[((size_t)w * p.chunk_rows + c) * p.topk + i];
                    }
            }
        };
        // this warp's Top-kappa lists start empty: (-inf, no id)
        float* const my_tv = tk_val + (size_t)q * p.chunk_rows * p.topk;
        int* const my_ti = tk_idx + (size_t)q * p.chunk_rows * p.topk;
        int ab = 0;
        uint32_t aph = 0;
        bool ok = true;
        // One row chunk: a CTA meets the same hidden rows in every unit and keeps a running state per row, flushed once
        // (one partial per CTA).  Several chunks: every unit flushes its own partial (one per 128-row vocabulary tile).
        const bool running = p.n_chunks == 1;
        if (kReduce && running) {
            for (int c = lane; c < kMaxChunkRows; c += 32) { my_max[c] = -INFINITY; my_idx[c] = 0x7fffffff; my_sum[c] = 0.f; }
            __syncwarp();
        }
        if constexpr (kReduce && kTopk) {
            for (int i = lane; i < p.chunk_rows * p.topk; i += 32) { my_tv[i] = -INFINITY; my_ti[i] = 0x7fffffff; }
            __syncwarp();
        }
        for (int u = pair; u < p.n_units; u += n_pairs) {
            int tile, slice, chunk;
            decode(u, tile, slice, chunk);
            const int rbase = chunk * p.chunk_rows;
            const int vt = tile * 2 + (int)rank;                 // 128-row vocabulary tile of this CTA
            if (ok && (ctrl->abort || !ptx::mbar_wait(&ctrl->acc_full[ab], aph, p.wait_limit))) { fail(p, ctrl, 16); ok = false; }
            if (ok) {
                ptx::tc_fence_after();
                // (a unit of fewer than 128 rows per CTA leaves stale shared memory in the accumulator lanes beyond them)
                const int vid = vt * p.rows_cta + q * 32 + lane;
                const bool valid = q * 32 + lane < p.rows_cta && vid < p.V;
                const bool any_valid = __ballot_sync(0xffffffffu, valid) != 0;          // warp-uniform
                const int n_rows = min(p.chunk_rows, p.M - rbase);                       // hidden rows of this chunk
                const float sw = (kFp8 && valid) ? p.w_scale[vid] : 1.f;                 // fp8: this lane's weight-row scale
                for (int cg = 0; cg < n_cg; ++cg) {
                    uint32_t r[32];
                    ptx::tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ab * p.acc_stride + cg * 32), r);
                    ptx::tmem_ld_wait();
                    float upd_m = -INFINITY, upd_s = 0.f;
                    int upd_i = 0x7fffffff;
                    const int ncol = n_rows - cg * 32;       // columns of this group that are hidden rows (the rest hold zeros)
                    if (any_valid && ncol > 0) {
                        // The 32 columns go through the reductions side by side (no branch inside, so the shuffle
                        // chains of different columns overlap); lane j keeps the result of column j.
                        float v[32], m[32];
                        if constexpr (kFp8) {
                            // logit = (sum of e4m3 products) * weight-row scale * hidden-row scale; lane j fetches column j's scale
                            const int cr = rbase + cg * 32 + lane;
                            const float sh = cr < p.M ? p.h_scale[cr] : 0.f;
#pragma unroll
                            for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * (sw * __shfl_sync(0xffffffffu, sh, j)));
                        }
#pragma unroll
                        for (int j = 0; j < 32; ++j) m[j] = v[j] = valid ? __uint_as_float(r[j]) : -INFINITY;
                        if (p.logits_out && valid) {
                            float* dst = p.logits_out + ((size_t)slice * p.M + rbase + cg * 32) * p.V + vid;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < ncol) dst[(size_t)j * p.V] = v[j];
                        }
                        if constexpr (kReduce && kTopk) {
                            // lane j owns column j's list.  Its last entry is the bar: which lanes hold a logit of column j that
                            // passes it?  (Nothing to do but for a few tiles.)
                            const int K = p.topk;
                            float* const lv = my_tv + (size_t)(cg * 32 + lane) * K;
                            int* const li = my_ti + (size_t)(cg * 32 + lane) * K;
                            const float bar_mine = lane < ncol ? lv[K - 1] : INFINITY;
                            unsigned myhit = 0;
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const float bar_j = __shfl_sync(0xffffffffu, bar_mine, j);
                                const unsigned hit = __ballot_sync(0xffffffffu, v[j] >= bar_j && v[j] > -INFINITY);
                                if (lane == j) myhit = hit;
                            }
                            // rounds: every owner takes the next lane of its mask; one shuffle per column fetches that logit
                            while (__any_sync(0xffffffffu, myhit != 0)) {
                                const int src = myhit ? __ffs(myhit) - 1 : 0;
                                const bool have = myhit != 0;
                                myhit &= myhit - 1;
                                float x = -INFINITY;
#pragma unroll
                                for (int j = 0; j < 32; ++j) {
                                    const float t = __shfl_sync(0xffffffffu, v[j], src);
                                    if (lane == j) x = t;
                                }
                                if (have) topk_list_insert(lv, li, K, x, vid - lane + src);
                            }
                            __syncwarp();
                        }
                        if (kReduce) {
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) m[j] = fmaxf(m[j], __shfl_xor_sync(0xffffffffu, m[j], o));
                        }
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const unsigned eq = __ballot_sync(0xffffffffu, v[j] == m[j]);
                            if (lane == j) { upd_m = m[j]; upd_i = vid - lane + (__ffs(eq) - 1); }
                            v[j] = exp2f((v[j] - m[j]) * p.inv_T_log2e);
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] += __shfl_xor_sync(0xffffffffu, v[j], o);
                        }
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (lane == j) upd_s = v[j];
                        }
                    }
                    const int c = cg * 32 + lane;          // lane j holds column cg*32+j of this unit
                    if (!kReduce) {
                    } else if (!running) {
                        my_max[c] = upd_m; my_idx[c] = upd_i; my_sum[c] = upd_s;
                    } else if (upd_m != -INFINITY) {
                        const float om = my_max[c], os = my_sum[c];
                        if (upd_m > om) {           // ids only grow along a CTA's units: equality keeps the older, lower id
                            my_sum[c] = upd_s + (om == -INFINITY ? 0.f : os * exp2f((om - upd_m) * p.inv_T_log2e));
                            my_max[c] = upd_m;
                            my_idx[c] = upd_i;
                        } else {
                            my_sum[c] = os + upd_s * exp2f((upd_m - om) * p.inv_T_log2e);
                        }
                    }
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_rank(&ctrl->acc_empty[ab], 0));
            }
            if (++ab == kAcc) { ab = 0; aph ^= 1; }
            if (kReduce && !running) {
                // fold the four warps' results (disjoint vocabulary rows) into one partial per hidden row
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (ok && !ctrl->abort) flush((size_t)vt * p.M, rbase);
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
        }
        if (kReduce && running) {
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (ok && !ctrl->abort) flush((size_t)blockIdx.x * p.M, 0);
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    cluster_sync_all();                 // no remote arrive or multicast commit is in flight towards a CTA that has left
    if (warp == 1) {
        ptx::tc_fence_after();
        tmem_dealloc_pair(tmem_base, (uint32_t)p.tmem_cols);
    }
}

__global__ void __launch_bounds__(kThreads, 2)
lmhead_pair_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_h, const PairParams p) {
    pair_gemm_body<true, false, false>(tm_w, tm_h, p);
}
__global__ void __launch_bounds__(kThreads, 2)
lmhead_pair_topk_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_h, const PairParams p) {
    pair_gemm_body<true, false, true>(tm_w, tm_h, p);
}
__global__ void __launch_bounds__(kThreads, 2)
lmhead_pair_fp8_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_h, const PairParams p) {
    pair_gemm_body<true, true, false>(tm_w, tm_h, p);
}
__global__ void __launch_bounds__(kThreads, 2)
linear_pair_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_h, const PairParams p) {
    pair_gemm_body<false, false, false>(tm_w, tm_h, p);
}

int next_pow2(int x) {
    int p = 1;
    while (p < x) p <<= 1;
    return p;
}

int ctas_per_sm_for(const MirrorTuning& tune, int M) {
    const int max_rows = tune.lm_pair2_max_rows;      // up to this many rows two CTAs share an SM (<= 256 TMEM columns and >= 4 stages each)
    int c = M <= max_rows ? 2 : 1;
    if (tune.lm_ctas_per_sm == 1 || (tune.lm_ctas_per_sm == 2 && M <= max_rows)) c = tune.lm_ctas_per_sm;
    return c;
}

// shapes shared by both modes: row chunks, accumulator layout, pipeline depth
mirror_status pair_shape(const MirrorTuning& tune, int M, int V, int H, PairParams* p, int rows_cta = kTileV, int topk = 0) {
    if (M <= 0 || V <= 0 || H <= 0 || H % kBK != 0) return MIRROR_ERR_SHAPE;
    p->M = M; p->V = V; p->H = H;
    p->n_chunks = (M + kMaxChunkRows - 1) / kMaxChunkRows;
    p->chunk_rows = (int)align_up((size_t)((M + p->n_chunks - 1) / p->n_chunks), 16);
    p->half_rows = p->chunk_rows / 2;
    p->acc_stride = next_pow2(p->chunk_rows < 32 ? 32 : p->chunk_rows);
    p->tmem_cols = kAcc * p->acc_stride;
    p->rows_cta = rows_cta;
    p->a_bytes = rows_cta * kBK * 2;
    p->stage_bytes = p->a_bytes + p->half_rows * kBK * 2;
    // Few rows (a weight stream): two CTAs per SM with five or six stages each keep more bytes in flight than one CTA with
    // eight, deal the units to twice as many pairs, and let the CTAs of the next kernel move in one by one.
    p->ctas_per_sm = ctas_per_sm_for(tune, M);
    p->topk = topk;
    p->topk_bytes = topk > 0 ? (int)align_up((size_t)4 * p->chunk_rows * (size_t)topk * 8, 256) : 0;
    p->part_topv = nullptr; p->part_topi = nullptr;
    if (p->topk_bytes > (32 << 10)) p->ctas_per_sm = 1;
    p->stages = (kSmemBudget / p->ctas_per_sm - kCtrlBytes - 2048 - p->topk_bytes) / p->stage_bytes;
    if (p->stages > kMaxStages) p->stages = kMaxStages;
    if (tune.lm_stages >= 2 && tune.lm_stages < p->stages) p->stages = tune.lm_stages;
    p->wait_limit = tune.wait_limit_cycles;
    p->stall_after = -1;
    if (p->stages < 2) return MIRROR_ERR_SHAPE;
    p->k_slices = 1;
    p->kb_per_slice = H / kBK;
    p->inv_T = p->inv_T_log2e = 1.f;
    p->logits_out = nullptr;
    p->fp8 = 0; p->w_scale = nullptr; p->h_scale = nullptr;
    p->part_max = nullptr; p->part_idx = nullptr; p->part_sum = nullptr;
    return MIRROR_OK;
}

mirror_status pair_launch(mirror_ctx* ctx, bool reduce, const void* x, const void* W, PairParams& p, int n_pairs, cudaStream_t stream) {
    CUtensorMap tm_w, tm_h;
    {
        const uint64_t dims[2] = {(uint64_t)p.H, (uint64_t)p.V};
        const uint64_t strides[1] = {(uint64_t)p.H * 2};
        const uint32_t box_w[2] = {kBK, (uint32_t)p.rows_cta};
        mirror_status st = mirror_make_tmap(ctx, &tm_w, W, 2, dims, strides, box_w);
        if (st != MIRROR_OK) return st;
        const uint64_t hdims[2] = {(uint64_t)p.H, (uint64_t)p.M};
        const uint32_t box_h[2] = {kBK, (uint32_t)p.half_rows};
        st = mirror_make_tmap(ctx, &tm_h, x, 2, hdims, strides, box_h);
        if (st != MIRROR_OK) return st;
    }
    const size_t smem = (size_t)p.stages * p.stage_bytes + kCtrlBytes + p.topk_bytes + 1024;
    if (!ctx->lm_pair_attr_set) {
        MIRROR_CUDA_OK(cudaFuncSetAttribute(lmhead_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
        MIRROR_CUDA_OK(cudaFuncSetAttribute(lmhead_pair_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
        MIRROR_CUDA_OK(cudaFuncSetAttribute(lmhead_pair_fp8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
        MIRROR_CUDA_OK(cudaFuncSetAttribute(linear_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
        ctx->lm_pair_attr_set = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_pairs * 2);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (p.fp8 && (p.topk > 0 || !reduce)) return MIRROR_ERR_UNSUPPORTED;
    auto kern = !reduce ? linear_pair_kernel : p.fp8 ? lmhead_pair_fp8_kernel : p.topk > 0 ? lmhead_pair_topk_kernel : lmhead_pair_kernel;
    MIRROR_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, tm_w, tm_h, p));
    ctx->launches += 1;
    MIRROR_CUDA_OK(cudaGetLastError());
    return MIRROR_OK;
}

}  // namespace

int mirror_lmhead_pair_partials(int V) { return 2 * ((V + kPairV - 1) / kPairV); }

bool mirror_lmhead_topk_fusable(const mirror_ctx* ctx, int M, int topk) {
    if (topk <= 0 || M > kMaxChunkRows || M < ctx->tune.lm_pair_min_rows) return false;
    const size_t bytes = (size_t)4 * align_up((size_t)M, 16) * (size_t)topk * 8;
    return bytes <= ((size_t)96 << 10);           // (beyond 32 KB the kernel runs one CTA per SM)
}

mirror_status mirror_lmhead_pair_launch(mirror_ctx* ctx, const void* hidden, int M, const void* W, float* logits_out,
                                        void* partial_ws, size_t partial_bytes, cudaStream_t stream, int* n_partials,
                                        const float* w_scale, const float* h_scale, int topk, void* topk_ws, size_t topk_ws_bytes) {
    const bool fp8 = w_scale != nullptr;
    if (fp8 && (!h_scale || ctx->desc.hidden % 128 != 0)) return MIRROR_ERR_SHAPE;
    // (e4m3 rows are staged exactly like bf16 rows of half as many elements: the same bytes, boxes and swizzle)
    const int V = ctx->desc.vocab, H = fp8 ? ctx->desc.hidden / 2 : ctx->desc.hidden;
    // A weight stream (two CTAs per SM) is as long as its busiest pair: the rows a CTA takes per unit are chosen so that
    // the units come out in whole waves over the pairs (152064 rows over 148 pairs: five units of 2 x 104 rows each
    // instead of four or five of 2 x 128).
    int rows_cta = kTileV;
    if (ctas_per_sm_for(ctx->tune, M) == 2) {
        const int pairs = ctx->num_sms;
        long long best = -1;
        for (int r = kTileV; r >= 64; r -= 8) {
            const long long units = (V + 2 * r - 1) / (2 * r), waves = (units + pairs - 1) / pairs;
            if (best < 0 || waves * r < best) { best = waves * r; rows_cta = r; }
        }
        if (ctx->tune.lm_rows >= 8 && ctx->tune.lm_rows <= kTileV && ctx->tune.lm_rows % 8 == 0) rows_cta = ctx->tune.lm_rows;
    }
    const int n_tiles = (V + 2 * rows_cta - 1) / (2 * rows_cta);
    PairParams p;
    mirror_status st = pair_shape(ctx->tune, M, V, H, &p, rows_cta, topk);
    if (st != MIRROR_OK) return st;
    p.n_units = n_tiles * p.n_chunks;
    int n_pairs = ctx->num_sms / 2 * p.ctas_per_sm;
    if (n_pairs > p.n_units) n_pairs = p.n_units;
    if (n_pairs < 1) return MIRROR_ERR_UNSUPPORTED;
    // partials: one per CTA (single row chunk: running state) or one per 128-row vocabulary tile
    const size_t P = p.n_chunks == 1 ? (size_t)2 * n_pairs : (size_t)2 * n_tiles;
    if (partial_bytes < P * M * 12) return MIRROR_ERR_WORKSPACE;
    p.w_keep = p.n_chunks > 1;
    if (ctx->tune.test_stall_after >= 0 && ctx->tune.test_stall_lm_left-- > 0) p.stall_after = ctx->tune.test_stall_after;
    p.inv_T = 1.0f / ctx->temperature;
    p.inv_T_log2e = p.inv_T * 1.4426950408889634f;
    p.logits_out = logits_out;
    p.part_max = (float*)partial_ws;
    p.part_idx = (int*)(p.part_max + P * M);
    p.part_sum = (float*)(p.part_idx + P * M);
    p.status = ctx->d_status;
    if (topk > 0) {
        // the lists live as long as the CTA: one row chunk only (and four lists per CTA and row have to fit beside the stages)
        if (p.n_chunks != 1 || p.stages < 3) return MIRROR_ERR_UNSUPPORTED;
        if (!topk_ws || topk_ws_bytes < 4 * P * M * (size_t)topk * 8) return MIRROR_ERR_WORKSPACE;
        p.part_topv = (float*)topk_ws;
        p.part_topi = (int*)(p.part_topv + 4 * P * M * (size_t)topk);
    }
    p.fp8 = fp8 ? 1 : 0;
    p.w_scale = w_scale;
    p.h_scale = h_scale;
    st = pair_launch(ctx, true, hidden, W, p, n_pairs, stream);
    if (st != MIRROR_OK) return st;
    *n_partials = (int)P;
    return MIRROR_OK;
}

// Split of the K axis for a plain GEMM with few output tiles: the slice count that fills the CTA pairs best (whole
// waves of units), slices of at least 512 K elements.
int mirror_linear_slices(const mirror_ctx* ctx, int M, int N, int K) {
    const int n_tiles = (N + kPairV - 1) / kPairV, n_chunks = (M + kMaxChunkRows - 1) / kMaxChunkRows;
    const int n_kb = K / kBK, n_pairs = ctx->num_sms / 2 > 0 ? ctx->num_sms / 2 * ctas_per_sm_for(ctx->tune, M) : 1;
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= 16; ++s) {
        const int per = (n_kb + s - 1) / s;
        if (s > 1 && per < 8) break;
        const int eff_s = (n_kb + per - 1) / per;
        const long long units = (long long)n_tiles * n_chunks * eff_s;
        const long long waves = (units + n_pairs - 1) / n_pairs;
        const double eff = (double)units / (double)(waves * n_pairs);
        if (eff > best_eff + 0.02) { best_eff = eff; best = eff_s; }
    }
    return best;
}

// partial[s][M][N] (fp32) = sum over K slice s of x[M, K] * W[N, K]^T; the caller sums the slices in order.
mirror_status mirror_linear_partial_launch(mirror_ctx* ctx, const void* x, int M, const void* W, int N, int K, float* partial,
                                           size_t partial_bytes, cudaStream_t stream, int* k_slices) {
    PairParams p;
    mirror_status st = pair_shape(ctx->tune, M, N, K, &p);
    if (st != MIRROR_OK) return st;
    const int n_tiles = (N + kPairV - 1) / kPairV, n_kb = K / kBK;
    const int s = mirror_linear_slices(ctx, M, N, K);
    p.kb_per_slice = (n_kb + s - 1) / s;
    p.k_slices = (n_kb + p.kb_per_slice - 1) / p.kb_per_slice;
    if (partial_bytes < (size_t)p.k_slices * M * N * sizeof(float)) return MIRROR_ERR_WORKSPACE;
    p.n_units = n_tiles * p.n_chunks * p.k_slices;
    int n_pairs = ctx->num_sms / 2 * p.ctas_per_sm;
    if (n_pairs > p.n_units) n_pairs = p.n_units;
    if (n_pairs < 1) return MIRROR_ERR_UNSUPPORTED;
    p.w_keep = p.n_chunks > 1;
    p.logits_out = partial;
    p.status = ctx->d_status;
    st = pair_launch(ctx, false, x, W, p, n_pairs, stream);
    if (st != MIRROR_OK) return st;
    *k_slices = p.k_slices;
    return MIRROR_OK;
}
