// Branch-tree attention of the verify step: every tree node (kappa x gamma draft tokens + the root)
// attends to the paged KV cache of the verified prefix and to the tree's own K/V under the
// branch-causal mask (node i sees tree token j iff j is i or an ancestor of i), for all layers.
//
// Work decomposition.  A "unit" is (layer, request, KV head): all G = Hq/Hkv query heads of all n tree
// nodes (G*n rows) share that head's K/V stream, so one CTA owning the unit's rows reads each K/V byte
// once from HBM and reuses it from shared memory for every row (the GQA / tree sharing).  A unit's keys
// are cut into 16-token slots (one KV page, or 16 tree tokens) and 64-token tiles.  The tiles of all
// units form one sequence that is split evenly over persistent CTAs (one per SM), so a unit may be cut
// across CTAs; each CTA then leaves a partial (max, sum, accumulator) and the last one to arrive at the
// unit's counter merges them in a fixed order.  No CTA ever waits for another.
// More than 128 rows per unit are handled by row blocks: a group of CTAs walks the same tiles at the
// same time, each with its own rows, so the second read of a tile is served by L2.
//
// Per CTA: warp 0 stages tiles (one 5-D TMA box per full KV page and tensor, 128-byte swizzle; ragged
// pages and tree tokens by plain loads with zero fill), warps 1..8 each own 16 rows: QK^T and PV on
// mma.sync.m16n8k16 (bf16 in, fp32 accumulate), mask applied to the score fragment in registers,
// online softmax with quad shuffles.
#include <math.h>
#include <string.h>

#include "mirror_internal.h"

namespace {

constexpr int kConsumerWarps = 7;     // 8 warps per CTA: two per SM sub-partition, so each thread may use up to 255 registers
constexpr int kThreads = 32 * (1 + kConsumerWarps);
constexpr int kSlotTok = 16;
constexpr int kTileSlots = 4;
constexpr int kTileTok = kSlotTok * kTileSlots;     // 64
constexpr int kMaxBatch = 1024;
constexpr int kStagesD128 = 5;

struct AttnTree {
    unsigned long long anc[MIRROR_MAX_NODES][2];
};

struct AttnParams {
    int L, B, n, Hq, Hkv, G;
    int rows, n_rb, rows_per_rb;          // rows per unit, row blocks, rows per block (multiple of 16)
    int n_groups;                         // CTA groups (grid = n_groups * n_rb)
    int max_pages, num_pages, layer_pages;
    int tree_slots;
    float scale_log2e, scale;
    const int32_t* page_table;
    const int32_t* prefix_len;
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_pool;
    const __nv_bfloat16* v_pool;
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    __nv_bfloat16* out;
    float* lse_out;
    float* partial;                       // [grid][2][128][D+2]
    int* ticket;                          // [units][n_rb][kConsumerWarps]
    int* status;
};

struct UnitPos {                          // where a global tile index falls
    int layer, b, g;
    int tile_in_unit, tiles_in_unit;
    long long unit_first_tile;            // global index of the unit's first tile
};

__device__ __forceinline__ void dev_check(const AttnParams& p, int detail) {
    if (atomicCAS(p.status, 0, MIRROR_DEV_CHECK) == 0) atomicExch(p.status + 1, detail);
}

__device__ __forceinline__ UnitPos locate(long long x, const AttnParams& p, const int* cumT, long long tiles_per_layer) {
    UnitPos u;
    u.layer = (int)(x / tiles_per_layer);
    const long long rem = x - (long long)u.layer * tiles_per_layer;
    int b = 0;
    while (b + 1 < p.B && (long long)p.Hkv * cumT[b + 1] <= rem) ++b;
    const int Tb = cumT[b + 1] - cumT[b];
    const long long r2 = rem - (long long)p.Hkv * cumT[b];
    u.b = b;
    u.g = (int)(r2 / Tb);
    u.tile_in_unit = (int)(r2 - (long long)u.g * Tb);
    u.tiles_in_unit = Tb;
    u.unit_first_tile = x - u.tile_in_unit;
    return u;
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int D>
struct Cfg {
    static constexpr int kSlotBytes = kSlotTok * D * 2;       // one tensor's 16-token slot
    static constexpr int kTileBytes = kTileSlots * kSlotBytes;
    static constexpr int kStageBytes = 2 * kTileBytes;        // K then V
    static constexpr int kStages = (D == 128) ? kStagesD128 : 8;
};

// byte offset of (token row `tr` of a slot, 16-byte column chunk `c`) inside one tensor's slot:
// [D/64][16 rows][128 B] with the 128-byte swizzle TMA applies (chunk index ^ row % 8)
__device__ __forceinline__ uint32_t slot_off(int tr, int c) {
    return (uint32_t)((c >> 3) * 2048 + tr * 128 + (((c & 7) ^ (tr & 7)) << 4));
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_verify_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ AttnTree tree, const AttnParams p) {
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* full = (uint64_t*)(smem + (size_t)C::kStages * C::kStageBytes);
    uint64_t* empty = full + C::kStages;
    int* cumT = (int*)(empty + C::kStages);                  // [B+1] tiles per request, prefix-summed
    int* s_len = cumT + (kMaxBatch + 1);                      // [B] clamped prefix lengths
    __shared__ volatile int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int group = blockIdx.x / p.n_rb, rb = blockIdx.x % p.n_rb;

    // ---- prologue: tiles per request ------------------------------------------------------------
    for (int b = tid; b < p.B; b += kThreads) {
        int len = p.prefix_len[b];
        if (len < 0 || len > p.max_pages * kSlotTok) { dev_check(p, 300 + b); len = len < 0 ? 0 : p.max_pages * kSlotTok; }
        s_len[b] = len;
    }
    if (tid == 0) {
        for (int s = 0; s < C::kStages; ++s) { ptx::mbar_init(&full[s], 2); ptx::mbar_init(&empty[s], kConsumerWarps); }
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tm_k);
        ptx::prefetch_tmap(&tm_v);
        s_abort = 0;
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        cumT[0] = 0;
        for (int b = 0; b < p.B; ++b) {
            const int slots = (s_len[b] + kSlotTok - 1) / kSlotTok + p.tree_slots;
            acc += (slots + kTileSlots - 1) / kTileSlots;
            cumT[b + 1] = acc;
        }
    }
    __syncthreads();
    const long long tiles_per_layer = (long long)p.Hkv * cumT[p.B];
    const long long total_tiles = tiles_per_layer * p.L;
    // never more groups than tiles, so that every group's range is non-empty and boundaries are distinct
    const int n_groups = (int)min((long long)p.n_groups, total_tiles);
    if (group >= n_groups) return;
    const long long x_begin = total_tiles * group / n_groups;
    const long long x_end = total_tiles * (group + 1) / n_groups;

    if (warp == 0) {
        // =========================================================================== producer
        long long it = 0;
        bool ok = true;
        long long x = x_begin;
        while (x < x_end && ok) {
            const UnitPos u = locate(x, p, cumT, tiles_per_layer);
            const int len = s_len[u.b];
            const int pages_full = len / kSlotTok, pages_all = (len + kSlotTok - 1) / kSlotTok;
            const int t_last = (int)min((long long)u.tiles_in_unit, (long long)u.tile_in_unit + (x_end - x));
            const int32_t* pt = p.page_table + (size_t)u.b * p.max_pages;
            for (int t = u.tile_in_unit; t < t_last && ok; ++t, ++it, ++x) {
                const int s = (int)(it % C::kStages);
                const uint32_t ph = (uint32_t)((it / C::kStages) & 1);
                bool w = true;
                if (lane == 0) w = !s_abort && ptx::mbar_wait(&empty[s], ph ^ 1);
                w = __shfl_sync(0xffffffffu, w, 0);
                if (!w) {
                    if (lane == 0) { s_abort = 1; if (atomicCAS(p.status, 0, MIRROR_DEV_TIMEOUT) == 0) atomicExch(p.status + 1, 10); }
                    ok = false;
                    break;
                }
                uint8_t* sk = smem + (size_t)s * C::kStageBytes;
                uint8_t* sv = sk + C::kTileBytes;
                if (lane == 0) ptx::fence_proxy_async();     // earlier plain stores to this stage precede the bulk copies
                // full pages by TMA
                int n_tma = 0;
#pragma unroll
                for (int j = 0; j < kTileSlots; ++j) n_tma += (t * kTileSlots + j < pages_full) ? 1 : 0;
                if (lane == 0) {
                    ptx::mbar_arrive_expect_tx(&full[s], (uint32_t)(n_tma * 2 * C::kSlotBytes));
                    for (int j = 0; j < n_tma; ++j) {
                        int page = pt[t * kTileSlots + j];
                        if (page < 0 || page >= p.num_pages) { dev_check(p, 400); page = 0; }
                        const int pg = u.layer * p.layer_pages + page;
                        ptx::tma_load_5d(sk + j * C::kSlotBytes, &tm_k, &full[s], 0, 0, 0, u.g, pg);
                        ptx::tma_load_5d(sv + j * C::kSlotBytes, &tm_v, &full[s], 0, 0, 0, u.g, pg);
                    }
                }
                // ragged page, tree tokens and empty slots by plain loads (rows beyond the valid count are zero)
                for (int j = n_tma; j < kTileSlots; ++j) {
                    const int sl = t * kTileSlots + j;
                    const __nv_bfloat16 *ksrc = nullptr, *vsrc = nullptr;
                    size_t row_stride = 0;
                    int valid = 0;
                    if (sl < pages_all) {
                        int page = pt[sl];
                        if (page < 0 || page >= p.num_pages) { if (lane == 0) dev_check(p, 401); page = 0; }
                        const size_t off = (((size_t)u.layer * p.layer_pages + page) * p.Hkv + u.g) * (size_t)(kSlotTok * D);
                        ksrc = p.k_pool + off; vsrc = p.v_pool + off;
                        row_stride = D;
                        valid = len - pages_full * kSlotTok;
                    } else if (sl < pages_all + p.tree_slots) {
                        const int j0 = (sl - pages_all) * kSlotTok;
                        const size_t off = ((((size_t)u.layer * p.B + u.b) * p.n + j0) * p.Hkv + u.g) * (size_t)D;
                        ksrc = p.k_new + off; vsrc = p.v_new + off;
                        row_stride = (size_t)p.Hkv * D;
                        valid = min(kSlotTok, p.n - j0);
                    }
                    constexpr int kChunks = kSlotTok * D / 8;          // 16-byte chunks per tensor slot
                    for (int c = lane; c < kChunks; c += 32) {
                        const int tr = c / (D / 8), cc = c % (D / 8);
                        uint4 kvv = make_uint4(0, 0, 0, 0), vvv = make_uint4(0, 0, 0, 0);
                        if (tr < valid) {
                            kvv = *reinterpret_cast<const uint4*>(ksrc + tr * row_stride + cc * 8);
                            vvv = *reinterpret_cast<const uint4*>(vsrc + tr * row_stride + cc * 8);
                        }
                        *reinterpret_cast<uint4*>(sk + j * C::kSlotBytes + slot_off(tr, cc)) = kvv;
                        *reinterpret_cast<uint4*>(sv + j * C::kSlotBytes + slot_off(tr, cc)) = vvv;
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&full[s]);
            }
        }
        if (!ok && lane == 0) {
            const long long first = it > C::kStages ? it - C::kStages : 0;
            for (long long j = first; j < it; ++j)
                ptx::mbar_wait(&full[j % C::kStages], (uint32_t)((j / C::kStages) & 1), 100000000ull);
        }
        return;
    }

    // =============================================================================== consumers
    const int cw = warp - 1;
    const int gq = lane >> 2, tq = lane & 3;
    const int rb_row0 = rb * p.rows_per_rb;
    const int rb_rows = min(p.rows_per_rb, p.rows - rb_row0);           // rows of this block that exist
    const int wrow0 = rb_row0 + cw * 16;                                 // first row (within the unit) of this warp
    const bool warp_active = cw * 16 < rb_rows;
    const int r_lo = wrow0 + gq, r_hi = wrow0 + gq + 8;                  // this thread's two rows
    const bool lo_ok = warp_active && (cw * 16 + gq) < rb_rows, hi_ok = warp_active && (cw * 16 + gq + 8) < rb_rows;
    const int node_lo = lo_ok ? r_lo / p.G : 0, node_hi = hi_ok ? r_hi / p.G : 0;
    const unsigned long long anc_lo0 = tree.anc[node_lo][0], anc_lo1 = tree.anc[node_lo][1];
    const unsigned long long anc_hi0 = tree.anc[node_hi][0], anc_hi1 = tree.anc[node_hi][1];
    const uint32_t smem_base = ptx::smem_u32(smem);

    long long it = 0;
    long long x = x_begin;
    bool ok = true;
    while (x < x_end && ok) {
        const UnitPos u = locate(x, p, cumT, tiles_per_layer);
        const int len = s_len[u.b];
        const int pages_full = len / kSlotTok, pages_all = (len + kSlotTok - 1) / kSlotTok;
        const int t_last = (int)min((long long)u.tiles_in_unit, (long long)u.tile_in_unit + (x_end - x));
        const bool whole_unit = (u.tile_in_unit == 0 && t_last == u.tiles_in_unit);

        // Q fragments of this warp's 16 rows (row r = node * G + local head)
        uint32_t qf[D / 16][4];
        {
            const size_t qbase = (((size_t)u.layer * p.B + u.b) * p.n) * (size_t)p.Hq * D;
            const __nv_bfloat16* qlo = p.q + qbase + ((size_t)node_lo * p.Hq + u.g * p.G + (lo_ok ? r_lo % p.G : 0)) * D;
            const __nv_bfloat16* qhi = p.q + qbase + ((size_t)node_hi * p.Hq + u.g * p.G + (hi_ok ? r_hi % p.G : 0)) * D;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const int c0 = ks * 16 + tq * 2;
                qf[ks][0] = lo_ok ? *reinterpret_cast<const uint32_t*>(qlo + c0) : 0u;
                qf[ks][1] = hi_ok ? *reinterpret_cast<const uint32_t*>(qhi + c0) : 0u;
                qf[ks][2] = lo_ok ? *reinterpret_cast<const uint32_t*>(qlo + c0 + 8) : 0u;
                qf[ks][3] = hi_ok ? *reinterpret_cast<const uint32_t*>(qhi + c0 + 8) : 0u;
            }
        }
        float o[D / 8][4];
#pragma unroll
        for (int i = 0; i < D / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
        float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

        for (int t = u.tile_in_unit; t < t_last; ++t, ++it, ++x) {
            const int s = (int)(it % C::kStages);
            const uint32_t ph = (uint32_t)((it / C::kStages) & 1);
            if (s_abort || !ptx::mbar_wait(&full[s], ph)) {
                if (lane == 0) { s_abort = 1; if (atomicCAS(p.status, 0, MIRROR_DEV_TIMEOUT) == 0) atomicExch(p.status + 1, 11); }
                ok = false;
                break;
            }
            if (warp_active) {
                const uint32_t sk = smem_base + (uint32_t)(s * C::kStageBytes);
                const uint32_t sv = sk + C::kTileBytes;
                // ---- S = Q K^T over the 64 tokens of the tile
                float sc[kTileTok / 8][4];
#pragma unroll
                for (int i = 0; i < kTileTok / 8; ++i) { sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f; }
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
                    for (int np = 0; np < kTileTok / 16; ++np) {
                        // lanes address: token = np*16 + (lane/16)*8 + lane%8 ; chunk = 2*ks + (lane/8)&1
                        const int tok = np * 16 + ((lane >> 4) << 3) + (lane & 7);
                        const int ch = 2 * ks + ((lane >> 3) & 1);
                        uint32_t b0, b1, b2, b3;
                        ldsm_x4(sk + (uint32_t)((tok >> 4) * C::kSlotBytes) + slot_off(tok & 15, ch), b0, b1, b2, b3);
                        mma_bf16(sc[2 * np], qf[ks], b0, b1);
                        mma_bf16(sc[2 * np + 1], qf[ks], b2, b3);
                    }
                }
                // ---- mask: only tiles that hold a ragged page, tree tokens or empty slots need it
                const bool special = (t * kTileSlots + kTileSlots > pages_full);
                if (special) {
#pragma unroll
                    for (int nt = 0; nt < kTileTok / 8; ++nt) {
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int tok = nt * 8 + tq * 2 + e;
                            const int sl = t * kTileSlots + (tok >> 4), tr = tok & 15;
                            bool vis_lo, vis_hi;
                            if (sl < pages_full) { vis_lo = vis_hi = true; }
                            else if (sl < pages_all) { vis_lo = vis_hi = (sl * kSlotTok + tr) < len; }
                            else if (sl < pages_all + p.tree_slots) {
                                const int j = (sl - pages_all) * kSlotTok + tr;
                                vis_lo = (j < 64) ? ((anc_lo0 >> j) & 1ull) : ((anc_lo1 >> (j - 64)) & 1ull);
                                vis_hi = (j < 64) ? ((anc_hi0 >> j) & 1ull) : ((anc_hi1 >> (j - 64)) & 1ull);
                                if (j >= p.n) vis_lo = vis_hi = false;
                            } else { vis_lo = vis_hi = false; }
                            if (!vis_lo) sc[nt][e] = -INFINITY;
                            if (!vis_hi) sc[nt][2 + e] = -INFINITY;
                        }
                    }
                }
                // ---- online softmax (scores are raw dot products; the scale is folded into exp2)
                float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
                for (int nt = 0; nt < kTileTok / 8; ++nt) {
                    mx_lo = fmaxf(mx_lo, fmaxf(sc[nt][0], sc[nt][1]));
                    mx_hi = fmaxf(mx_hi, fmaxf(sc[nt][2], sc[nt][3]));
                }
                mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
                mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
                mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
                mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
                const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
                const float a_lo = (m_lo == -INFINITY) ? 0.f : exp2f((m_lo - mn_lo) * p.scale_log2e);
                const float a_hi = (m_hi == -INFINITY) ? 0.f : exp2f((m_hi - mn_hi) * p.scale_log2e);
                const float ms_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo * p.scale_log2e;
                const float ms_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi * p.scale_log2e;
                m_lo = mn_lo; m_hi = mn_hi;
                float sum_lo = 0.f, sum_hi = 0.f;
                uint32_t pf[kTileTok / 16][4];
#pragma unroll
                for (int nt = 0; nt < kTileTok / 8; ++nt) {
                    const float p0 = exp2f(fmaf(sc[nt][0], p.scale_log2e, -ms_lo));
                    const float p1 = exp2f(fmaf(sc[nt][1], p.scale_log2e, -ms_lo));
                    const float p2 = exp2f(fmaf(sc[nt][2], p.scale_log2e, -ms_hi));
                    const float p3 = exp2f(fmaf(sc[nt][3], p.scale_log2e, -ms_hi));
                    sum_lo += p0 + p1; sum_hi += p2 + p3;
                    pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
                    pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
                }
                l_lo = l_lo * a_lo + sum_lo;
                l_hi = l_hi * a_hi + sum_hi;
#pragma unroll
                for (int i = 0; i < D / 8; ++i) { o[i][0] *= a_lo; o[i][1] *= a_lo; o[i][2] *= a_hi; o[i][3] *= a_hi; }
                // ---- O += P V
#pragma unroll
                for (int ks = 0; ks < kTileTok / 16; ++ks) {
#pragma unroll
                    for (int np = 0; np < D / 16; ++np) {
                        // lanes address: token = ks*16 + ((lane/8)&1)*8 + lane%8 ; chunk = 2*np + lane/16
                        const int tok = ks * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);
                        const int ch = 2 * np + (lane >> 4);
                        uint32_t b0, b1, b2, b3;
                        ldsm_x4_t(sv + (uint32_t)((tok >> 4) * C::kSlotBytes) + slot_off(tok & 15, ch), b0, b1, b2, b3);
                        mma_bf16(o[2 * np], pf[ks], b0, b1);
                        mma_bf16(o[2 * np + 1], pf[ks], b2, b3);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&empty[s]);
        }
        if (!ok) break;
        if (!warp_active) continue;

        // row sums across the quad
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

        const size_t obase = (((size_t)u.layer * p.B + u.b) * p.n) * (size_t)p.Hq * D;
        __nv_bfloat16* olo = p.out + obase + ((size_t)node_lo * p.Hq + u.g * p.G + (lo_ok ? r_lo % p.G : 0)) * D;
        __nv_bfloat16* ohi = p.out + obase + ((size_t)node_hi * p.Hq + u.g * p.G + (hi_ok ? r_hi % p.G : 0)) * D;
        float* lse_lo = p.lse_out ? p.lse_out + (((size_t)u.layer * p.B + u.b) * p.Hq + u.g * p.G + (lo_ok ? r_lo % p.G : 0)) * p.n + node_lo : nullptr;
        float* lse_hi = p.lse_out ? p.lse_out + (((size_t)u.layer * p.B + u.b) * p.Hq + u.g * p.G + (hi_ok ? r_hi % p.G : 0)) * p.n + node_hi : nullptr;

        if (whole_unit) {
            const float inv_lo = 1.f / l_lo, inv_hi = 1.f / l_hi;
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                if (lo_ok) *reinterpret_cast<uint32_t*>(olo + i * 8 + tq * 2) = pack_bf16(o[i][0] * inv_lo, o[i][1] * inv_lo);
                if (hi_ok) *reinterpret_cast<uint32_t*>(ohi + i * 8 + tq * 2) = pack_bf16(o[i][2] * inv_hi, o[i][3] * inv_hi);
            }
            if (lse_lo && tq == 0) {
                if (lo_ok) *lse_lo = m_lo * p.scale + logf(l_lo);
                if (hi_ok) *lse_hi = m_hi * p.scale + logf(l_hi);
            }
            continue;
        }

        // ---- the unit is cut across CTA groups: leave a partial, last arrival merges ----------------
        // groups ga..gb cover this unit (group g owns tiles [total*g/n_groups, total*(g+1)/n_groups))
        const long long per = total_tiles;
        int ga = group, gb = group;
        while (ga > 0 && per * ga / n_groups > u.unit_first_tile) --ga;
        const long long unit_last = u.unit_first_tile + u.tiles_in_unit - 1;
        while (gb + 1 < n_groups && per * (gb + 1) / n_groups <= unit_last) ++gb;
        const int parts = gb - ga + 1;
        const int slot = (u.tile_in_unit > 0) ? 0 : 1;      // a unit that began before this CTA's range uses slot 0
        constexpr int kRowW = D + 2;
        float* my = p.partial + (((size_t)blockIdx.x * 2 + slot) * 128 + cw * 16) * kRowW;
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            *reinterpret_cast<float2*>(my + (size_t)gq * kRowW + i * 8 + tq * 2) = make_float2(o[i][0], o[i][1]);
            *reinterpret_cast<float2*>(my + (size_t)(gq + 8) * kRowW + i * 8 + tq * 2) = make_float2(o[i][2], o[i][3]);
        }
        if (tq == 0) {
            my[(size_t)gq * kRowW + D] = m_lo; my[(size_t)gq * kRowW + D + 1] = l_lo;
            my[(size_t)(gq + 8) * kRowW + D] = m_hi; my[(size_t)(gq + 8) * kRowW + D + 1] = l_hi;
        }
        __threadfence();
        __syncwarp();
        const size_t unit_idx = ((size_t)u.layer * p.B + u.b) * p.Hkv + u.g;
        int* tk = p.ticket + (unit_idx * p.n_rb + rb) * kConsumerWarps + cw;
        int arrived = 0;
        if (lane == 0) arrived = atomicAdd(tk, 1);
        arrived = __shfl_sync(0xffffffffu, arrived, 0);
        if (arrived != parts - 1) continue;
        __threadfence();
        if (lane == 0) *tk = 0;                              // ready for the next launch
        // merge in group order
        float M_lo = -INFINITY, M_hi = -INFINITY;
        for (int gsrc = ga; gsrc <= gb; ++gsrc) {
            const int sslot = (per * gsrc / n_groups > u.unit_first_tile) ? 0 : 1;
            const float* src = p.partial + (((size_t)(gsrc * p.n_rb + rb) * 2 + sslot) * 128 + cw * 16) * kRowW;
            M_lo = fmaxf(M_lo, __ldcg(src + (size_t)gq * kRowW + D));
            M_hi = fmaxf(M_hi, __ldcg(src + (size_t)(gq + 8) * kRowW + D));
        }
        float L_lo = 0.f, L_hi = 0.f;
#pragma unroll
        for (int i = 0; i < D / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
        for (int gsrc = ga; gsrc <= gb; ++gsrc) {
            const int sslot = (per * gsrc / n_groups > u.unit_first_tile) ? 0 : 1;
            const float* src = p.partial + (((size_t)(gsrc * p.n_rb + rb) * 2 + sslot) * 128 + cw * 16) * kRowW;
            const float pm_lo = __ldcg(src + (size_t)gq * kRowW + D), pm_hi = __ldcg(src + (size_t)(gq + 8) * kRowW + D);
            const float w_lo = (pm_lo == -INFINITY) ? 0.f : exp2f((pm_lo - M_lo) * p.scale_log2e);
            const float w_hi = (pm_hi == -INFINITY) ? 0.f : exp2f((pm_hi - M_hi) * p.scale_log2e);
            L_lo += w_lo * __ldcg(src + (size_t)gq * kRowW + D + 1);
            L_hi += w_hi * __ldcg(src + (size_t)(gq + 8) * kRowW + D + 1);
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                const float2 vlo = __ldcg(reinterpret_cast<const float2*>(src + (size_t)gq * kRowW + i * 8 + tq * 2));
                const float2 vhi = __ldcg(reinterpret_cast<const float2*>(src + (size_t)(gq + 8) * kRowW + i * 8 + tq * 2));
                o[i][0] += w_lo * vlo.x; o[i][1] += w_lo * vlo.y;
                o[i][2] += w_hi * vhi.x; o[i][3] += w_hi * vhi.y;
            }
        }
        const float inv_lo = 1.f / L_lo, inv_hi = 1.f / L_hi;
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            if (lo_ok) *reinterpret_cast<uint32_t*>(olo + i * 8 + tq * 2) = pack_bf16(o[i][0] * inv_lo, o[i][1] * inv_lo);
            if (hi_ok) *reinterpret_cast<uint32_t*>(ohi + i * 8 + tq * 2) = pack_bf16(o[i][2] * inv_hi, o[i][3] * inv_hi);
        }
        if (lse_lo && tq == 0) {
            if (lo_ok) *lse_lo = M_lo * p.scale + logf(L_lo);
            if (hi_ok) *lse_hi = M_hi * p.scale + logf(L_hi);
        }
    }
}

}  // namespace

mirror_status mirror_attn_launch(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const MirrorTreeInfo& ti,
                                 const void* q, const void* k_new, const void* v_new, void* out, float* lse_out,
                                 float* partial_ws, int* ticket_ws, size_t ticket_ints, cudaStream_t stream) {
    const int D = ctx->desc.head_dim, Hkv = ctx->desc.n_kv_heads, Hq = ctx->desc.n_q_heads;
    AttnParams p;
    p.L = kv->num_layers; p.B = tree->batch; p.n = ti.n; p.Hq = Hq; p.Hkv = Hkv; p.G = Hq / Hkv;
    p.rows = p.G * p.n;
    p.n_rb = (p.rows + kConsumerWarps * 16 - 1) / (kConsumerWarps * 16);
    p.rows_per_rb = (int)align_up((size_t)((p.rows + p.n_rb - 1) / p.n_rb), 16);
    p.n_groups = ctx->num_sms / p.n_rb;
    if (p.n_groups < 1) return MIRROR_ERR_SHAPE;
    p.max_pages = kv->max_pages_per_req; p.num_pages = kv->num_pages;
    const int64_t page_elems = (int64_t)Hkv * kSlotTok * D;
    if (kv->layer_stride % page_elems != 0) return MIRROR_ERR_UNSUPPORTED;
    p.layer_pages = (int)(kv->layer_stride / page_elems);
    p.tree_slots = (p.n + kSlotTok - 1) / kSlotTok;
    p.scale = ctx->scale;
    p.scale_log2e = ctx->scale * 1.4426950408889634f;
    p.page_table = kv->page_table; p.prefix_len = kv->prefix_len;
    p.q = (const __nv_bfloat16*)q;
    p.k_pool = (const __nv_bfloat16*)kv->k_pool; p.v_pool = (const __nv_bfloat16*)kv->v_pool;
    p.k_new = (const __nv_bfloat16*)k_new; p.v_new = (const __nv_bfloat16*)v_new;
    p.out = (__nv_bfloat16*)out; p.lse_out = lse_out;
    p.partial = partial_ws; p.ticket = ticket_ws; p.status = ctx->d_status;
    if ((size_t)p.L * p.B * Hkv * p.n_rb * kConsumerWarps > ticket_ints) return MIRROR_ERR_WORKSPACE;
    if (p.B > kMaxBatch) return MIRROR_ERR_SHAPE;

    AttnTree at;
    memcpy(at.anc, ti.anc, sizeof at.anc);

    CUtensorMap tm_k, tm_v;
    {
        const uint64_t total_pages = (uint64_t)(p.L - 1) * p.layer_pages + p.num_pages;
        const uint64_t dims[5] = {64, (uint64_t)kSlotTok, (uint64_t)(D / 64), (uint64_t)Hkv, total_pages};
        const uint64_t strides[4] = {(uint64_t)D * 2, 128, (uint64_t)kSlotTok * D * 2, (uint64_t)page_elems * 2};
        const uint32_t box[5] = {64, (uint32_t)kSlotTok, (uint32_t)(D / 64), 1, 1};
        mirror_status st = mirror_make_tmap(ctx, &tm_k, kv->k_pool, 5, dims, strides, box);
        if (st != MIRROR_OK) return st;
        st = mirror_make_tmap(ctx, &tm_v, kv->v_pool, 5, dims, strides, box);
        if (st != MIRROR_OK) return st;
    }
    const int grid = p.n_groups * p.n_rb;
    if (D == 128) {
        using C = Cfg<128>;
        const size_t smem = (size_t)C::kStages * C::kStageBytes + 2 * C::kStages * 8 + (2 * kMaxBatch + 2) * 4 + 1024;
        MIRROR_CUDA_OK(cudaFuncSetAttribute(attn_verify_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attn_verify_kernel<128><<<grid, kThreads, smem, stream>>>(tm_k, tm_v, at, p);
    } else {
        using C = Cfg<64>;
        const size_t smem = (size_t)C::kStages * C::kStageBytes + 2 * C::kStages * 8 + (2 * kMaxBatch + 2) * 4 + 1024;
        MIRROR_CUDA_OK(cudaFuncSetAttribute(attn_verify_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attn_verify_kernel<64><<<grid, kThreads, smem, stream>>>(tm_k, tm_v, at, p);
    }
    ctx->launches += 1;
    MIRROR_CUDA_OK(cudaGetLastError());
    return MIRROR_OK;
}
