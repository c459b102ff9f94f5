// LM head logits = W h (Eq. 1; early-exit proxy Eq. 5): what surrounds the GEMM (dispatch, merge of the row partials,
// Top-kappa of Eq. 6, gathers, the public entry points) and the single-CTA GEMM kernel.  The GEMM normally runs on CTA
// pairs (lmhead_pair.cu); lmhead_kernel below is the one-CTA-per-SM version that serves when the scratch a caller gave
// cannot hold the pair kernel's partials.  Both fuse the per-row argmax / max / log-sum-exp reduction into the
// epilogue, so that the [M, V] logits never travel through HBM unless the caller asks for them (speculative sampling,
// Top-kappa).
//
// lmhead_kernel, orientation ("swap-AB"): the vocabulary is the UMMA M axis (128 weight rows per tile, one TMEM
// lane per vocabulary id), the hidden rows are the UMMA N axis (<= 256 per chunk, one TMEM column
// per hidden row).  The verify step has few rows (B * (1 + kappa*gamma)), so the kernel is a weight
// stream: W leaves HBM exactly once per row chunk and the per-SM TMA pipeline is what has to keep
// HBM busy.
//
// Persistent CTAs, one per SM, 6 warps:
//   warp 0      TMA producer: W tile [128 x 64] + hidden tile [N x 64] per stage, 128-byte swizzle
//   warp 1      TMEM owner and UMMA issuer (one elected lane): 4 x (128 x N x 16) per stage
//   warps 2..5  epilogue: tcgen05.ld the accumulator (lane = vocabulary id), per-column warp
//               reductions, running (max, argmax, sum-exp) per hidden row, optional fp32 spill
// The vocabulary is split over CTAs in 8-row groups (the swizzle atom), so every CTA streams the same
// number of weight bytes (+-8 rows); the ragged last tile of a CTA is fetched as 8-row TMA boxes.
// Each CTA leaves one partial per hidden row; lmhead_merge_kernel merges them in a
// fixed order with the comparator (logit descending, id ascending).
//
// Every mbarrier wait is bounded; on expiry the kernel records MIRROR_DEV_TIMEOUT and unwinds.
#include <math.h>
#include <stdlib.h>

#include <mutex>

#include <cuda_fp8.h>

#include "mirror_internal.h"

namespace {

constexpr int kThreads = 192;
constexpr int kBK = 64;                 // K elements per pipeline stage (one 128-byte swizzle row)
constexpr int kTileV = 128;             // vocabulary rows per UMMA tile
constexpr int kATileBytes = kTileV * kBK * 2;
constexpr int kMaxStages = 10;
constexpr int kMaxAcc = 4;
constexpr int kMaxChunkRows = 256;
constexpr int kSmemBudget = 232448;     // 227 KB
constexpr int kCtrlBytes = 1024 + 4 * kMaxChunkRows * 12;   // barriers + per-warp running state

struct LmParams {
    int M, V, H;
    int n_chunks, chunk_rows;           // hidden rows are processed in chunks of chunk_rows (multiple of 16)
    int acc_stride, n_acc, tmem_cols;   // TMEM columns per accumulator buffer, number of buffers, allocation
    int stages, stage_bytes;
    int k_group;                        // producer batching: K blocks requested together
    int groups_total;                   // ceil(V / 8)
    float inv_T, inv_T_log2e;
    float* logits_out;                  // nullable [M, V]
    float* part_max;                    // [grid][M]
    int* part_idx;
    float* part_sum;
    int* status;
    long long wait_limit;               // SM cycles after which a wait gives up
};

struct Ctrl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t acc_full[kMaxAcc];
    uint64_t acc_empty[kMaxAcc];
    uint32_t tmem_base;
    volatile int abort;
};

__device__ __forceinline__ void fail(const LmParams& p, Ctrl* c, int where) {
    c->abort = 1;
    if (atomicCAS(p.status, 0, MIRROR_DEV_TIMEOUT) == 0) atomicExch(p.status + 1, where);
}

__global__ void __launch_bounds__(kThreads, 1)
lmhead_kernel(const __grid_constant__ CUtensorMap tm_w_full, const __grid_constant__ CUtensorMap tm_w_grp,
              const __grid_constant__ CUtensorMap tm_h, const LmParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_base = smem;
    Ctrl* ctrl = (Ctrl*)(smem + (size_t)p.stages * p.stage_bytes);
    float* st_max = (float*)((uint8_t*)ctrl + 1024);          // [4][kMaxChunkRows]
    int* st_idx = (int*)(st_max + 4 * kMaxChunkRows);
    float* st_sum = (float*)(st_idx + 4 * kMaxChunkRows);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // this CTA's slice of the vocabulary, in 8-row groups
    const int g0 = (int)(((long long)p.groups_total * blockIdx.x) / gridDim.x);
    const int g1 = (int)(((long long)p.groups_total * (blockIdx.x + 1)) / gridDim.x);
    const int row_begin = g0 * 8;
    const int row_end = min(g1 * 8, p.V);
    const int n_tiles = (g1 - g0 + 15) / 16;
    const int n_kb = p.H / kBK;

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) { ptx::mbar_init(&ctrl->full[s], 1); ptx::mbar_init(&ctrl->empty[s], 1); }
        for (int a = 0; a < p.n_acc; ++a) { ptx::mbar_init(&ctrl->acc_full[a], 1); ptx::mbar_init(&ctrl->acc_empty[a], 4); }
        ctrl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tm_w_full);
        ptx::prefetch_tmap(&tm_w_grp);
        ptx::prefetch_tmap(&tm_h);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&ctrl->tmem_base, (uint32_t)p.tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    // (programmatic dependent launch: the set-up above overlaps the kernel ahead in the stream; nothing of global
    // memory is touched before it has completed)
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint64_t pol_w = ptx::policy_evict_first();
            const uint64_t pol_h = ptx::policy_evict_last();
            const uint32_t b_bytes = (uint32_t)p.chunk_rows * kBK * 2;
            // pipeline position kept as (stage, phase) counters: this single thread is on the critical path
            // and 64-bit divisions by a run-time stage count would cost more than the copies it issues
            int s0 = 0;                 // stage of the next K block to issue
            uint32_t ph0 = 0;           // its phase bit
            int issued = 0;
            bool ok = true;
            for (int chunk = 0; chunk < p.n_chunks && ok; ++chunk)
                for (int t = 0; t < n_tiles && ok; ++t) {
                    const int row0 = row_begin + t * kTileV;
                    const int ng = min(16, g1 - (g0 + t * 16));
                    const uint32_t tx_bytes = (uint32_t)ng * 1024u + b_bytes;
                    // K blocks are issued in batches of k_group so that the copies that touch one DRAM page
                    // (consecutive 128-byte pieces of one weight row) are requested together instead of one
                    // pipeline stage apart.
                    for (int kb0 = 0; kb0 < n_kb && ok; kb0 += p.k_group) {
                        const int nk = min(p.k_group, n_kb - kb0);
                        {
                            int s = s0;
                            uint32_t ph = ph0;
                            for (int j = 0; j < nk; ++j) {
                                if (ctrl->abort || !ptx::mbar_wait(&ctrl->empty[s], ph ^ 1, p.wait_limit)) { fail(p, ctrl, 1); ok = false; break; }
                                ptx::mbar_arrive_expect_tx(&ctrl->full[s], tx_bytes);
                                if (++s == p.stages) { s = 0; ph ^= 1; }
                            }
                        }
                        if (!ok) break;
                        // (the tensor maps are named directly: a pointer chosen at run time would make the compiler
                        // copy the kernel parameters to local memory)
                        if (ng == 16) {
                            int s = s0;
                            for (int j = 0; j < nk; ++j) {
                                ptx::tma_load_2d_hint(stage_base + s * p.stage_bytes, &tm_w_full, &ctrl->full[s],
                                                      (kb0 + j) * kBK, row0, pol_w);
                                if (++s == p.stages) s = 0;
                            }
                        } else {
                            for (int g = 0; g < ng; ++g) {
                                int s = s0;
                                for (int j = 0; j < nk; ++j) {
                                    ptx::tma_load_2d_hint(stage_base + s * p.stage_bytes + g * 1024, &tm_w_grp, &ctrl->full[s],
                                                          (kb0 + j) * kBK, row0 + g * 8, pol_w);
                                    if (++s == p.stages) s = 0;
                                }
                            }
                        }
                        for (int j = 0; j < nk; ++j) {
                            ptx::tma_load_2d_hint(stage_base + s0 * p.stage_bytes + kATileBytes, &tm_h, &ctrl->full[s0],
                                                  (kb0 + j) * kBK, chunk * p.chunk_rows, pol_h);
                            if (++s0 == p.stages) { s0 = 0; ph0 ^= 1; }
                        }
                        issued += nk;
                    }
                }
            if (!ok) {
                // let copies already in flight land before the CTA's shared memory goes away
                const int back = issued < p.stages ? issued : p.stages;
                int s = s0;
                uint32_t ph = ph0;
                for (int j = 0; j < back; ++j) {
                    if (--s < 0) { s = p.stages - 1; ph ^= 1; }
                    ptx::mbar_wait(&ctrl->full[s], ph, 200000000ll);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ UMMA issuer
        if (lane == 0) {
            const uint32_t idesc = ptx::umma_idesc_bf16(kTileV, p.chunk_rows);
            const uint32_t stage_u32 = ptx::smem_u32(stage_base);
            int s = 0, ab = 0;
            uint32_t ph = 0, aph = 0;
            bool ok = true;
            for (int chunk = 0; chunk < p.n_chunks && ok; ++chunk)
                for (int t = 0; t < n_tiles && ok; ++t) {
                    if (ctrl->abort || !ptx::mbar_wait(&ctrl->acc_empty[ab], aph ^ 1, p.wait_limit)) { fail(p, ctrl, 2); ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)(ab * p.acc_stride);
                    for (int kb = 0; kb < n_kb; ++kb) {
                        if (ctrl->abort || !ptx::mbar_wait(&ctrl->full[s], ph, p.wait_limit)) { fail(p, ctrl, 3); ok = false; break; }
                        ptx::tc_fence_after();
                        const uint32_t sa = stage_u32 + (uint32_t)(s * p.stage_bytes);
                        const uint32_t sb = sa + kATileBytes;
#pragma unroll
                        for (int k4 = 0; k4 < kBK / 16; ++k4)
                            ptx::umma_f16(d_tmem, ptx::umma_desc_k_sw128(sa + k4 * 32), ptx::umma_desc_k_sw128(sb + k4 * 32),
                                          idesc, (kb | k4) != 0);
                        ptx::umma_commit(&ctrl->empty[s]);
                        if (++s == p.stages) { s = 0; ph ^= 1; }
                    }
                    if (ok) ptx::umma_commit(&ctrl->acc_full[ab]);
                    if (++ab == p.n_acc) { ab = 0; aph ^= 1; }
                }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        float* my_max = st_max + q * kMaxChunkRows;
        int* my_idx = st_idx + q * kMaxChunkRows;
        float* my_sum = st_sum + q * kMaxChunkRows;
        const int n_cg = (p.chunk_rows + 31) / 32;
        int ab = 0;
        uint32_t aph = 0;
        bool ok = true;
        for (int chunk = 0; chunk < p.n_chunks; ++chunk) {
            const int rbase = chunk * p.chunk_rows;
            for (int c = lane; c < kMaxChunkRows; c += 32) { my_max[c] = -INFINITY; my_idx[c] = 0x7fffffff; my_sum[c] = 0.f; }
            __syncwarp();
            for (int t = 0; t < n_tiles && ok; ++t) {
                if (ctrl->abort || !ptx::mbar_wait(&ctrl->acc_full[ab], aph, p.wait_limit)) { fail(p, ctrl, 4); ok = false; break; }
                ptx::tc_fence_after();
                const int vid = row_begin + t * kTileV + q * 32 + lane;      // this thread's vocabulary id
                const bool valid = vid < row_end;
                for (int cg = 0; cg < n_cg; ++cg) {
                    uint32_t r[32];
                    ptx::tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ab * p.acc_stride + cg * 32), r);
                    ptx::tmem_ld_wait();
                    float upd_m = -INFINITY, upd_s = 0.f;
                    int upd_i = 0x7fffffff;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int row = rbase + cg * 32 + j;
                        if (cg * 32 + j >= p.chunk_rows || row >= p.M) break;      // warp-uniform
                        const float v = valid ? __uint_as_float(r[j]) : -INFINITY;
                        if (p.logits_out && valid) p.logits_out[(size_t)row * p.V + vid] = v;
                        float m = v;
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                        if (m == -INFINITY) continue;                               // warp-uniform
                        const unsigned eq = __ballot_sync(0xffffffffu, v == m);
                        float e = exp2f((v - m) * p.inv_T_log2e);
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
                        if (lane == j) { upd_m = m; upd_s = e; upd_i = vid - lane + (__ffs(eq) - 1); }
                    }
                    // lane j folds column cg*32+j of this tile into the running state
                    const int c = cg * 32 + lane;
                    if (upd_m != -INFINITY) {
                        const float om = my_max[c], os = my_sum[c];
                        if (upd_m > om) {           // ids only grow along a CTA's tiles: equality keeps the older, lower id
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
                if (lane == 0) ptx::mbar_arrive(&ctrl->acc_empty[ab]);
                if (++ab == p.n_acc) { ab = 0; aph ^= 1; }
            }
            // fold the four warps' states (disjoint vocabulary rows) into one partial per hidden row
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (ok && !ctrl->abort) {
                const size_t pbase = (size_t)blockIdx.x * p.M;
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
                }
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// Merge the per-CTA partials of each hidden row: one block per row, one partial per thread, fixed
// reduction tree; the comparator (logit descending, id ascending) makes the result order-independent.
__global__ void __launch_bounds__(256)
lmhead_merge_kernel(int M, int P, float inv_T, float inv_T_log2e, const float* part_max, const int* part_idx,
                    const float* part_sum, int32_t* argmax, float* maxlogit, float* lse) {
    __shared__ float s_m[8], s_s[8];
    __shared__ int s_i[8];
    const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    float m = -INFINITY, s = 0.f;
    int idx = 0x7fffffff;
    auto fold = [&](float om, int oi, float os) {
        if (om == -INFINITY) return;
        if (om > m || (om == m && oi < idx)) {
            s = os + (m == -INFINITY ? 0.f : s * exp2f((m - om) * inv_T_log2e));
            m = om; idx = oi;
        } else {
            s += os * exp2f((om - m) * inv_T_log2e);
        }
    };
    for (int k = tid; k < P; k += blockDim.x)
        fold(part_max[(size_t)k * M + row], part_idx[(size_t)k * M + row], part_sum[(size_t)k * M + row]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, o), os = __shfl_xor_sync(0xffffffffu, s, o);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        fold(om, oi, os);
    }
    if (lane == 0) { s_m[warp] = m; s_i[warp] = idx; s_s[warp] = s; }
    __syncthreads();
    if (tid == 0) {
        m = -INFINITY; s = 0.f; idx = 0x7fffffff;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) fold(s_m[w], s_i[w], s_s[w]);
        if (argmax) argmax[row] = idx;
        if (maxlogit) maxlogit[row] = m;
        if (lse) lse[row] = m * inv_T + logf(s);
    }
}

// Top-kappa of each row (Eq. 6): k rounds of "best element strictly after the previous pick" in the order (logit
// descending, id ascending).  One block per row.  Either over the row's fp32 logits (cand_id == nullptr: V values, the
// id is the position), or over the candidate lists that the GEMM's epilogue left: n_part lists of list_k (logit, id)
// pairs per row, laid out [partial][row][list_k] (empty places hold -inf).
__global__ void __launch_bounds__(1024, 1)
lmhead_topk_kernel(int V, int topk, float inv_T, const float* logits, const float* lse, int32_t* topk_id,
                   float* topk_logprob, __nv_bfloat16* topk_logprob_bf16, const int* cand_id, int M, int list_k) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    __shared__ float s_v[32];
    __shared__ int s_i[32];
    __shared__ float s_prev_v;
    __shared__ int s_prev_i;
    const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* l = logits + (size_t)row * (cand_id ? list_k : V);
    const int* li = cand_id ? cand_id + (size_t)row * list_k : nullptr;
    const size_t part_stride = (size_t)M * list_k;                 // candidates: from one partial's list to the next
    if (tid == 0) { s_prev_v = INFINITY; s_prev_i = -1; }
    __syncthreads();
    for (int k = 0; k < topk; ++k) {
        const float pv = s_prev_v;
        const int pi = s_prev_i;
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int n = tid; n < V; n += blockDim.x) {
            float x;
            int v = n;
            if (li) {
                const size_t at = (size_t)(n / list_k) * part_stride + (size_t)(n % list_k);
                x = l[at];
                v = li[at];
            } else {
                x = l[n];
            }
            const bool after = (x < pv) || (x == pv && v > pi);
            if (after && (x > bv || (x == bv && v < bi))) { bv = x; bi = v; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) { s_v[warp] = bv; s_i[warp] = bi; }
        __syncthreads();
        if (warp == 0) {
            bv = s_v[lane]; bi = s_i[lane];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            if (lane == 0) {
                s_prev_v = bv; s_prev_i = bi;
                topk_id[(size_t)row * topk + k] = bi;
                const float lp = bv * inv_T - lse[row];
                if (topk_logprob) topk_logprob[(size_t)row * topk + k] = lp;
                if (topk_logprob_bf16) topk_logprob_bf16[(size_t)row * topk + k] = __float2bfloat16_rn(lp);      // token-channel payload
            }
        }
        __syncthreads();
    }
}

// logits[row][tok] for a short list of (row, token) pairs: one warp per pair, fp32 dot product.
__global__ void lmhead_gather_kernel(int n_gather, int M, int V, int H, const __nv_bfloat16* hidden,
                                     const __nv_bfloat16* W, const int32_t* gather_row, const int32_t* gather_tok,
                                     float* gather_logit, int* status) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const int g = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (g >= n_gather) return;
    const int row = gather_row[g], tok = gather_tok[g];
    if (row < 0 || row >= M || tok < 0 || tok >= V) {
        if (lane == 0) {
            gather_logit[g] = __int_as_float(0x7fc00000);
            if (atomicCAS(status, 0, MIRROR_DEV_CHECK) == 0) atomicExch(status + 1, 200);
        }
        return;
    }
    const __nv_bfloat162* h2 = (const __nv_bfloat162*)(hidden + (size_t)row * H);
    const __nv_bfloat162* w2 = (const __nv_bfloat162*)(W + (size_t)tok * H);
    float acc = 0.f;
    for (int k = lane; k < H / 2; k += 32) {
        const float2 a = __bfloat1622float2(h2[k]), b = __bfloat1622float2(w2[k]);
        acc = fmaf(a.x, b.x, acc);
        acc = fmaf(a.y, b.y, acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) gather_logit[g] = acc;
}

int next_pow2(int x) {
    int p = 1;
    while (p < x) p <<= 1;
    return p;
}

// What follows the GEMM, whichever kernel ran it: merge of the row partials, Top-kappa, gathers.
mirror_status lmhead_tail(mirror_ctx* ctx, const void* hidden, int M, const void* W, int topk, const int32_t* gather_row,
                          const int32_t* gather_tok, int n_gather, int32_t* argmax, float* maxlogit, float* lse, int32_t* topk_id,
                          float* topk_logprob, float* gather_logit, float* logits_out, float* lse_scratch, cudaStream_t stream,
                          void* topk_logprob_bf16, int P, float inv_T, float inv_T_log2e, const float* part_max, const int* part_idx,
                          const float* part_sum, const float* cand_v = nullptr, const int* cand_i = nullptr) {
    const int V = ctx->desc.vocab, H = ctx->desc.hidden;
    float* lse_dst = lse ? lse : (topk > 0 ? lse_scratch : nullptr);
    if (argmax || maxlogit || lse_dst) {
        MIRROR_CUDA_OK(mirror_launch_pdl(lmhead_merge_kernel, dim3(M), dim3(256), 0, stream, M, P, inv_T, inv_T_log2e,
                                         part_max, part_idx, part_sum, argmax, maxlogit, lse_dst));
        ctx->launches += 1;
        MIRROR_CUDA_OK(cudaGetLastError());
    }
    if (topk > 0) {
        if (cand_v)      // (four lists per partial: one per epilogue warp)
            MIRROR_CUDA_OK(mirror_launch_pdl(lmhead_topk_kernel, dim3(M), dim3(1024), 0, stream, 4 * P * topk, topk, inv_T, cand_v, lse_dst,
                                             topk_id, topk_logprob, (__nv_bfloat16*)topk_logprob_bf16, cand_i, M, topk));
        else
            MIRROR_CUDA_OK(mirror_launch_pdl(lmhead_topk_kernel, dim3(M), dim3(1024), 0, stream, V, topk, inv_T, (const float*)logits_out,
                                             lse_dst, topk_id, topk_logprob, (__nv_bfloat16*)topk_logprob_bf16, (const int*)nullptr, M, 0));
        ctx->launches += 1;
        MIRROR_CUDA_OK(cudaGetLastError());
    }
    if (n_gather > 0) {
        const int warps = 8;
        lmhead_gather_kernel<<<(n_gather + warps - 1) / warps, warps * 32, 0, stream>>>(
            n_gather, M, V, H, (const __nv_bfloat16*)hidden, (const __nv_bfloat16*)W, gather_row, gather_tok, gather_logit,
            ctx->d_status);
        ctx->launches += 1;
        MIRROR_CUDA_OK(cudaGetLastError());
    }
    return MIRROR_OK;
}

}  // namespace

mirror_status mirror_lmhead_launch(mirror_ctx* ctx, const void* hidden, int M, const void* W, int topk,
                                   const int32_t* gather_row, const int32_t* gather_tok, int n_gather,
                                   int32_t* argmax, float* maxlogit, float* lse, int32_t* topk_id,
                                   float* topk_logprob, float* gather_logit, float* logits_out,
                                   void* partial_ws, size_t partial_bytes, float* lse_scratch, cudaStream_t stream,
                                   cudaEvent_t after_gemm, void* topk_logprob_bf16, void* topk_ws, size_t topk_ws_bytes) {
    const int V = ctx->desc.vocab, H = ctx->desc.hidden;
    // Top-kappa inside the GEMM's epilogue whenever the caller's scratch holds the candidate lists; otherwise (or on the
    // single-CTA fallback kernel) the selection runs over spilled logits, which then have to be there.
    const bool fused_topk = topk > 0 && topk_ws != nullptr;
    if (topk > 0 && !fused_topk && !logits_out) return MIRROR_ERR_WORKSPACE;
    // The GEMM runs on CTA pairs (lmhead_pair.cu) whenever the partials it leaves fit the scratch it was given; the
    // single-CTA weight-stream kernel below is the fallback (and what MIRROR_LM_PAIR_MIN_ROWS can force for comparison).
    const int pair_min_rows = ctx->tune.lm_pair_min_rows;
    if (M >= pair_min_rows && ctx->num_sms >= 2) {
        int P = 0;
        mirror_status st = mirror_lmhead_pair_launch(ctx, hidden, M, W, logits_out, partial_ws, partial_bytes, stream, &P, nullptr,
                                                     nullptr, fused_topk ? topk : 0, topk_ws, topk_ws_bytes);
        if (st == MIRROR_OK) {
            if (after_gemm) MIRROR_CUDA_OK(cudaEventRecord(after_gemm, stream));
            const float inv_T = 1.0f / ctx->temperature, inv_T_log2e = inv_T * 1.4426950408889634f;
            float* part_max = (float*)partial_ws;
            int* part_idx = (int*)(part_max + (size_t)P * M);
            float* part_sum = (float*)(part_idx + (size_t)P * M);
            return lmhead_tail(ctx, hidden, M, W, topk, gather_row, gather_tok, n_gather, argmax, maxlogit, lse, topk_id, topk_logprob,
                               gather_logit, logits_out, lse_scratch, stream, topk_logprob_bf16, P, inv_T, inv_T_log2e, part_max,
                               part_idx, part_sum, fused_topk ? (const float*)topk_ws : nullptr,
                               fused_topk ? (const int*)((const float*)topk_ws + (size_t)4 * P * M * topk) : nullptr);
        }
        if (st != MIRROR_ERR_WORKSPACE) return st;
    }
    if (topk > 0 && !logits_out) return MIRROR_ERR_WORKSPACE;       // the single-CTA kernel selects from spilled logits only
    LmParams p;
    p.M = M; p.V = V; p.H = H;
    p.n_chunks = (M + kMaxChunkRows - 1) / kMaxChunkRows;
    p.chunk_rows = (int)align_up((size_t)((M + p.n_chunks - 1) / p.n_chunks), 16);
    p.acc_stride = next_pow2(p.chunk_rows < 32 ? 32 : p.chunk_rows);
    p.n_acc = 512 / p.acc_stride < kMaxAcc ? 512 / p.acc_stride : kMaxAcc;
    p.tmem_cols = p.n_acc * p.acc_stride;
    p.stage_bytes = kATileBytes + p.chunk_rows * kBK * 2;
    p.stages = (kSmemBudget - kCtrlBytes - 1024) / p.stage_bytes;
    if (p.stages > kMaxStages) p.stages = kMaxStages;
    if (p.stages < 2) return MIRROR_ERR_SHAPE;
    // producer batching (tuning knobs; the defaults were picked by measurement on B200)
    p.k_group = p.stages / 2 < 5 ? (p.stages / 2 > 0 ? p.stages / 2 : 1) : 5;
    if (ctx->tune.lm_kgroup > 0) p.k_group = ctx->tune.lm_kgroup;
    if (ctx->tune.lm_stages >= 2 && ctx->tune.lm_stages < p.stages) p.stages = ctx->tune.lm_stages;
    if (p.k_group < 1) p.k_group = 1;
    if (p.k_group > p.stages) p.k_group = p.stages;
    p.groups_total = (V + 7) / 8;
    p.inv_T = 1.0f / ctx->temperature;
    p.inv_T_log2e = p.inv_T * 1.4426950408889634f;
    p.logits_out = logits_out;
    p.status = ctx->d_status;
    p.wait_limit = ctx->tune.wait_limit_cycles;

    int grid = ctx->num_sms;
    if (grid > p.groups_total) grid = p.groups_total;
    const size_t P = (size_t)grid;
    if (partial_bytes < P * M * 12) return MIRROR_ERR_WORKSPACE;
    p.part_max = (float*)partial_ws;
    p.part_idx = (int*)(p.part_max + P * M);
    p.part_sum = (float*)(p.part_idx + P * M);

    CUtensorMap tm_w_full, tm_w_grp, tm_h;
    {
        const uint64_t dims[2] = {(uint64_t)H, (uint64_t)V};
        const uint64_t strides[1] = {(uint64_t)H * 2};
        const uint32_t box_full[2] = {kBK, kTileV}, box_grp[2] = {kBK, 8};
        mirror_status st = mirror_make_tmap(ctx, &tm_w_full, W, 2, dims, strides, box_full);
        if (st != MIRROR_OK) return st;
        st = mirror_make_tmap(ctx, &tm_w_grp, W, 2, dims, strides, box_grp);
        if (st != MIRROR_OK) return st;
        const uint64_t hdims[2] = {(uint64_t)H, (uint64_t)M};
        const uint32_t box_h[2] = {kBK, (uint32_t)p.chunk_rows};
        st = mirror_make_tmap(ctx, &tm_h, hidden, 2, hdims, strides, box_h);
        if (st != MIRROR_OK) return st;
    }
    const size_t smem = (size_t)p.stages * p.stage_bytes + kCtrlBytes + 1024;
    if (!ctx->lm_attr_set) {
        MIRROR_CUDA_OK(cudaFuncSetAttribute(lmhead_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
        ctx->lm_attr_set = true;
    }
    MIRROR_CUDA_OK(mirror_launch_pdl(lmhead_kernel, dim3(grid), dim3(kThreads), smem, stream, tm_w_full, tm_w_grp, tm_h, p));
    ctx->launches += 1;
    MIRROR_CUDA_OK(cudaGetLastError());
    if (after_gemm) MIRROR_CUDA_OK(cudaEventRecord(after_gemm, stream));

    return lmhead_tail(ctx, hidden, M, W, topk, gather_row, gather_tok, n_gather, argmax, maxlogit, lse, topk_id, topk_logprob,
                       gather_logit, logits_out, lse_scratch, stream, topk_logprob_bf16, (int)P, p.inv_T, p.inv_T_log2e, p.part_max,
                       p.part_idx, p.part_sum);
}

extern "C" mirror_status mirror_lmhead_reduce(mirror_ctx* ctx, const void* hidden, int M, const void* W, int topk,
                                              const int32_t* gather_row, const int32_t* gather_tok, int n_gather,
                                              int32_t* argmax, float* maxlogit, float* lse, int32_t* topk_id,
                                              float* topk_logprob, float* gather_logit, float* logits_out,
                                              void* stream) {
    if (!ctx || !hidden || !W || M <= 0 || topk < 0 || n_gather < 0) return MIRROR_ERR_ARG;
    if (topk > MIRROR_MAX_TOPK || topk > ctx->desc.vocab) return MIRROR_ERR_SHAPE;
    if (topk > 0 && (!topk_id || !topk_logprob)) return MIRROR_ERR_ARG;
    if (n_gather > 0 && (!gather_row || !gather_tok || !gather_logit)) return MIRROR_ERR_ARG;
    if (((uintptr_t)hidden & 15) || ((uintptr_t)W & 15)) return MIRROR_ERR_ARG;
    if (!ctx->ws) return MIRROR_ERR_WORKSPACE;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    MirrorWsLayout L;
    mirror_ws_layout(ctx, (size_t)M, &L);
    size_t need = L.end_lmhead;
    float* lse_scratch = (float*)((uint8_t*)ctx->ws + L.lse);
    void* topk_ws = nullptr;
    if (topk > 0) {
        if (L.lm_topk_bytes && ctx->ws_bytes >= L.end_topk && mirror_lmhead_topk_fusable(ctx, M, topk)) {
            topk_ws = (uint8_t*)ctx->ws + L.lm_topk;       // Top-kappa inside the GEMM's epilogue: no [M, V] buffer
            need = L.end_topk;
        } else if (!logits_out) {
            logits_out = (float*)((uint8_t*)ctx->ws + L.logits);
            need = L.end_logits;
        }
    }
    if (ctx->ws_bytes < need) return MIRROR_ERR_WORKSPACE;
    return mirror_lmhead_launch(ctx, hidden, M, W, topk, gather_row, gather_tok, n_gather, argmax, maxlogit, lse, topk_id,
                                topk_logprob, gather_logit, logits_out, (uint8_t*)ctx->ws + L.lm_partial, L.lm_partial_bytes, lse_scratch,
                                (cudaStream_t)stream, nullptr, nullptr, topk_ws, L.lm_topk_bytes);
}

// ---------------------------------------------------------------------------------------------------
// Low-precision LM head: W and the hidden rows as e4m3 bytes with one fp32 scale per row (W ~ w_scale[v] * W8[v, :],
// h ~ h_scale[r] * h8[r, :]); the GEMM runs on kind::f8f6f4 tensor-core instructions (fp32 accumulation of exact e4m3
// products) and the epilogue multiplies each accumulator by the two scales before the row reductions.  Half the weight
// bytes of the bf16 head: the weight stream of a verify step with few rows takes half the time.
// ---------------------------------------------------------------------------------------------------
namespace {

// one block per row: scale = max|x| / 448 (1 for an all-zero row), code = e4m3(x / scale), round to nearest even
__global__ void __launch_bounds__(256) quantize_rows_e4m3_kernel(const __nv_bfloat16* x, int cols, uint8_t* out, float* scale) {
    __shared__ float s_part[8];
    __shared__ float s_scale;
    const __nv_bfloat16* row = x + (size_t)blockIdx.x * cols;
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    float amax = 0.f;
    for (int c = threadIdx.x; c < cols; c += 256) amax = fmaxf(amax, fabsf(__bfloat162float(row[c])));
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float a = 0.f;
        for (int w = 0; w < 8; ++w) a = fmaxf(a, s_part[w]);
        const float sc = a > 0.f ? __fdiv_rn(a, 448.f) : 1.f;
        s_scale = sc;
        scale[blockIdx.x] = sc;
    }
    __syncthreads();
    const float sc = s_scale;
    uint8_t* dst = out + (size_t)blockIdx.x * cols;
    for (int c = threadIdx.x; c < cols; c += 256)
        dst[c] = (uint8_t)__nv_cvt_float_to_fp8(__fdiv_rn(__bfloat162float(row[c]), sc), __NV_SATFINITE, __NV_E4M3);
}

}  // namespace

extern "C" mirror_status mirror_quantize_rows_fp8(mirror_ctx* ctx, const void* x, int rows, int cols, void* out_fp8,
                                                  float* out_scale, void* stream) {
    if (!ctx || !x || !out_fp8 || !out_scale || rows <= 0 || cols <= 0) return MIRROR_ERR_ARG;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    MIRROR_CUDA_OK(mirror_launch_pdl(quantize_rows_e4m3_kernel, dim3((unsigned)rows), dim3(256), 0, (cudaStream_t)stream,
                                     (const __nv_bfloat16*)x, cols, (uint8_t*)out_fp8, out_scale));
    ctx->launches += 1;
    MIRROR_CUDA_OK(cudaGetLastError());
    return MIRROR_OK;
}

extern "C" mirror_status mirror_lmhead_reduce_fp8(mirror_ctx* ctx, const void* hidden_fp8, const float* h_scale, int M,
                                                  const void* W_fp8, const float* w_scale, int32_t* argmax, float* maxlogit,
                                                  float* lse, float* logits_out, void* stream) {
    if (!ctx || !hidden_fp8 || !h_scale || !W_fp8 || !w_scale || M <= 0) return MIRROR_ERR_ARG;
    if (((uintptr_t)hidden_fp8 & 15) || ((uintptr_t)W_fp8 & 15)) return MIRROR_ERR_ARG;
    if (ctx->desc.hidden % 128 != 0) return MIRROR_ERR_SHAPE;          // K in 128-byte blocks
    if (!ctx->ws) return MIRROR_ERR_WORKSPACE;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    MirrorWsLayout L;
    mirror_ws_layout(ctx, (size_t)M, &L);
    if (ctx->ws_bytes < L.end_lmhead) return MIRROR_ERR_WORKSPACE;
    void* partial_ws = (uint8_t*)ctx->ws + L.lm_partial;
    int P = 0;
    mirror_status st = mirror_lmhead_pair_launch(ctx, hidden_fp8, M, W_fp8, logits_out, partial_ws, L.lm_partial_bytes,
                                                 (cudaStream_t)stream, &P, w_scale, h_scale);
    if (st != MIRROR_OK) return st;
    const float inv_T = 1.0f / ctx->temperature, inv_T_log2e = inv_T * 1.4426950408889634f;
    float* part_max = (float*)partial_ws;
    int* part_idx = (int*)(part_max + (size_t)P * M);
    float* part_sum = (float*)(part_idx + (size_t)P * M);
    return lmhead_tail(ctx, nullptr, M, nullptr, 0, nullptr, nullptr, 0, argmax, maxlogit, lse, nullptr, nullptr, nullptr, logits_out,
                       nullptr, (cudaStream_t)stream, nullptr, P, inv_T, inv_T_log2e, part_max, part_idx, part_sum);
}

// ---------------------------------------------------------------------------------------------------
// mirror_lmhead_reduce_noalloc: the same LM-head kernels for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need the LM head: a
// serving loop that has handed all device memory to its own pool, a plugin running inside a framework's
// allocator-guarded region, or code that must not touch the allocator because a stream capture is
// under way elsewhere in the process.  For them the per-CTA partials (the kernel's only scratch memory)
// live in a fixed array that is part of the loaded library image, and no context object (whose
// creation allocates a status word) is needed.
// ---------------------------------------------------------------------------------------------------
namespace {

constexpr int kNoAllocMaxRows = 128;      // M limit of the no-allocation entry point
constexpr int kNoAllocMaxCtas = 320;      // partials of one launch: up to two CTAs on each of 160 SMs (a B200 has 148)
constexpr size_t kNoAllocHeader = 256;    // {status code, detail} words in front of the partials
constexpr size_t kNoAllocBytes = kNoAllocHeader + (size_t)kNoAllocMaxCtas * kNoAllocMaxRows * 12;

// Lives in every GPU's copy of the library image from load until exit (491,776 bytes per device).
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

struct NoAllocDevice {          // host-side, per device, filled by the first call on that device
    bool ready = false;
    unsigned char* scratch = nullptr;
    int num_sms = 0;
    bool attr_set = false, pair_attr_set = false;
    PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
};
NoAllocDevice g_noalloc_dev[64];
std::mutex g_noalloc_mutex;      // the one-time set-up of a device, and its `ready` flag, from any host thread

}  // namespace

extern "C" mirror_status mirror_lmhead_reduce_noalloc(int device, const void* hidden, int M, const void* W, int V, int H,
                                                      float temperature, int32_t* argmax, float* maxlogit, float* lse,
                                                      void* stream) {
    if (!hidden || !W || M <= 0 || V <= 0 || H <= 0 || device < 0 || device >= 64) return MIRROR_ERR_ARG;
    if (M > kNoAllocMaxRows) return MIRROR_ERR_SHAPE;          // beyond the fixed scratch: use mirror_lmhead_reduce
    if (H % 64 != 0 || temperature < 0.f) return MIRROR_ERR_SHAPE;
    if (((uintptr_t)hidden & 15) || ((uintptr_t)W & 15)) return MIRROR_ERR_ARG;
    MIRROR_CUDA_OK(cudaSetDevice(device));
    NoAllocDevice& d = g_noalloc_dev[device];
    std::unique_lock<std::mutex> lock(g_noalloc_mutex);
    if (!d.ready) {
        // one-time set-up on this device (no allocation): resolve the device address of the scratch array
        cudaDeviceProp prop;
        MIRROR_CUDA_OK(cudaGetDeviceProperties(&prop, device));
        if (prop.major != 10) return MIRROR_ERR_UNSUPPORTED;
        if (2 * prop.multiProcessorCount > kNoAllocMaxCtas) return MIRROR_ERR_UNSUPPORTED;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return MIRROR_ERR_CUDA;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
            qres != cudaDriverEntryPointSuccess)
            return MIRROR_ERR_CUDA;
        d.scratch = (unsigned char*)ptr;
        d.num_sms = prop.multiProcessorCount;
        d.encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
        d.ready = true;
    }
    lock.unlock();
    // A context on the stack stands in for mirror_create's: same launch path, nothing allocated.
    mirror_ctx tmp;
    tmp.desc.hidden = H;
    tmp.desc.vocab = V;
    tmp.desc.n_q_heads = tmp.desc.n_kv_heads = 1;
    tmp.desc.head_dim = 64;
    tmp.desc.page_size = 16;
    tmp.desc.softmax_scale = 0.f;
    tmp.desc.temperature = temperature;
    tmp.device = device;
    tmp.num_sms = d.num_sms;
    tmp.temperature = temperature > 0.f ? temperature : 1.0f;
    tmp.d_status = (int*)d.scratch;
    tmp.encode = d.encode;
    tmp.lm_attr_set = d.attr_set;
    tmp.lm_pair_attr_set = d.pair_attr_set;
    cudaStream_t s = (cudaStream_t)stream;
    // (the status words in the header start at zero with the library image and keep the first problem until
    // mirror_lmhead_noalloc_status reads and clears them; the partials are fully rewritten by every launch before
    // they are read)
    mirror_status st = mirror_lmhead_launch(&tmp, hidden, M, W, 0, nullptr, nullptr, 0, argmax, maxlogit, lse, nullptr, nullptr,
                                            nullptr, nullptr, d.scratch + kNoAllocHeader, kNoAllocBytes - kNoAllocHeader,
                                            nullptr, s, nullptr);
    d.attr_set = tmp.lm_attr_set;
    d.pair_attr_set = tmp.lm_pair_attr_set;
    return st;
}

// Device-side problems of mirror_lmhead_reduce_noalloc calls (a bounded wait that ran out, a failed bounds check) are
// recorded in the first words of the scratch array, since there is no context to ask.  Synchronises the device, returns
// the first problem since the last query (0: none) and clears it.  Allocates nothing.
extern "C" mirror_status mirror_lmhead_noalloc_status(int device, int* code, int* detail) {
    if (!code || device < 0 || device >= 64) return MIRROR_ERR_ARG;
    unsigned char* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (g_noalloc_dev[device].ready) scratch = g_noalloc_dev[device].scratch;
    }
    *code = 0;
    if (detail) *detail = 0;
    if (!scratch) return MIRROR_OK;                      // no call was ever made on this device
    MIRROR_CUDA_OK(cudaSetDevice(device));
    MIRROR_CUDA_OK(cudaDeviceSynchronize());
    int words[2] = {0, 0};
    MIRROR_CUDA_OK(cudaMemcpy(words, scratch, sizeof words, cudaMemcpyDeviceToHost));
    if (words[0] != 0) MIRROR_CUDA_OK(cudaMemset(scratch, 0, sizeof words));
    *code = words[0] == MIRROR_DEV_TIMEOUT ? MIRROR_ERR_TIMEOUT : (words[0] != 0 ? MIRROR_ERR_DEVICE_CHECK : MIRROR_OK);
    if (detail) *detail = words[1];
    return MIRROR_OK;
}
