// Branch-tree attention of the verify step: every tree node (kappa x gamma draft tokens + the root)
// attends to the paged KV cache of the verified prefix and to the tree's own K/V under the
// branch-causal mask (node i sees tree token j iff j is i or an ancestor of i), for all layers.
//
// Work decomposition.  A "unit" is (layer, request, KV head): all G = Hq/Hkv query heads of all n tree
// nodes (G*n rows) share that head's K/V stream, so one CTA owning the unit's rows reads each K/V byte
// once from HBM and reuses it from shared memory for every row (the GQA / tree sharing).  A unit's keys
// are cut into 16-token slots (one KV page, or 16 tree tokens) and 128-token tiles.  The tiles of all
// units form one sequence that is split evenly over persistent CTAs (one per SM), so a unit may be cut
// across CTAs; each CTA then leaves a partial (max, sum, accumulator) and the last one to arrive at the
// unit's counter merges them in a fixed order.  No CTA ever waits for another.
// More than 128 rows per unit are handled by row blocks: a group of CTAs walks the same tiles at the
// same time, each with its own rows, so the second read of a tile is served by L2.
//
// Per CTA (6 warps):
//   warp 0      stages K and V tiles: one TMA box per (page, 64-column half) issued by separate lanes,
//               128-byte swizzle; ragged page and tree tokens by plain loads with zero fill
//   warp 1      owns TMEM and issues tcgen05.mma: S = Q K^T (M=128 rows, N=tokens of the tile) into one of
//               two S buffers, then O += P V with P read from shared memory and V as an MN-major operand
//   warps 2..5  one thread per row (TMEM lane): tcgen05.ld of the row's scores, mask in registers, online
//               softmax without any shuffle, P written as bf16 into the swizzled A-operand layout; the
//               accumulator O stays in TMEM and is rescaled only when a row's maximum grew by more than
//               2^8 (the stale offset is carried exactly through the running sum and the final division)
// Every mbarrier wait is bounded; on expiry the kernel records MIRROR_DEV_TIMEOUT and unwinds.
#include <math.h>
#include <string.h>

#include "mirror_internal.h"

namespace {

constexpr int kThreads = 192;
constexpr int kSlotTok = 16;
constexpr int kTileSlots = 8;
constexpr int kTileTok = kSlotTok * kTileSlots;     // 128
constexpr int kRows = 128;                          // UMMA M: rows per row block
constexpr int kMaxBatch = 1024;
constexpr int kKVStages = 2;
constexpr int kMergeWarps = 4;
constexpr float kRescaleLog2 = 8.0f;

struct AttnTree {
    unsigned long long anc[MIRROR_MAX_NODES][2];
};

struct AttnParams {
    int L, B, n, Hq, Hkv, G;
    int rows, n_rb, rows_per_rb;          // rows per unit, row blocks, rows per block
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
    int* ticket;                          // [units][n_rb][kMergeWarps]
    int* status;
};

struct UnitPos {                          // where a global tile index falls
    int layer, b, g;
    int tile_in_unit, tiles_in_unit;
    long long unit_first_tile;            // global index of the unit's first tile
};

struct Ctrl {
    uint64_t k_full[kKVStages], k_empty[kKVStages], v_full[kKVStages], v_empty[kKVStages];
    uint64_t s_full[2], s_free[2];
    uint64_t q_full, p_full, pv_done;
    uint32_t tmem_base;
    volatile int abort;
};

__device__ __forceinline__ void dev_check(const AttnParams& p, int detail) {
    if (atomicCAS(p.status, 0, MIRROR_DEV_CHECK) == 0) atomicExch(p.status + 1, detail);
}
__device__ __forceinline__ void timeout(const AttnParams& p, Ctrl* c, int where) {
    c->abort = 1;
    if (atomicCAS(p.status, 0, MIRROR_DEV_TIMEOUT) == 0) atomicExch(p.status + 1, where);
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

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Shared-memory operand tiles are [64-column half][row][128 B] with the 128-byte swizzle: the 16-byte chunk
// index is XORed with (row % 8).  A half holds 128 rows = 16 KB.
constexpr int kHalfBytes = 128 * 128;
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {      // chunk: 16-byte column chunk, 0 .. D/8-1
    return (uint32_t)((chunk >> 3) * kHalfBytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// MN-major B operand (V: rows = tokens along K, 64 d-columns contiguous): 8-token groups 1024 B apart,
// 64-column halves kHalfBytes apart.
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);
    d |= (uint64_t)(kHalfBytes >> 4) << 16;          // leading byte offset: next 64-column atom
    d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset: next 8-token group
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

__device__ __forceinline__ void tmem_st_32x32b_x32(uint32_t taddr, const uint32_t (&r)[32]) {
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
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

template <int D>
struct Cfg {
    static constexpr int kHalves = D / 64;
    static constexpr int kOperandBytes = kHalves * kHalfBytes;     // a 128-row operand tile (Q, one K stage, one V stage)
    static constexpr int kPBytes = 2 * kHalfBytes;                 // P: 128 rows x 128 tokens
    static constexpr int kSlotBoxBytes = kSlotTok * 128;           // one TMA box: 16 tokens x 64 columns
    static constexpr size_t kSmemData = (size_t)kOperandBytes * (1 + 2 * kKVStages) + kPBytes;
    static constexpr size_t kSmemBytes = kSmemData + 1024 /*ctrl*/ + (2 * kMaxBatch + 2) * 4 + 1024 /*align*/;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_verify_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ AttnTree tree, const AttnParams p) {
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem;
    uint8_t* sP = sQ + C::kOperandBytes;
    uint8_t* sK = sP + C::kPBytes;                                  // [kKVStages]
    uint8_t* sV = sK + kKVStages * C::kOperandBytes;                // [kKVStages]
    Ctrl* ctrl = (Ctrl*)(sV + kKVStages * C::kOperandBytes);
    int* cumT = (int*)((uint8_t*)ctrl + 1024);                      // [B+1] tiles per request, prefix-summed
    int* s_len = cumT + (kMaxBatch + 1);                            // [B] clamped prefix lengths

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int group = blockIdx.x / p.n_rb, rb = blockIdx.x % p.n_rb;

    // ---- prologue ---------------------------------------------------------------------------------
    for (int b = tid; b < p.B; b += kThreads) {
        int len = p.prefix_len[b];
        if (len < 0 || len > p.max_pages * kSlotTok) { dev_check(p, 300 + b); len = len < 0 ? 0 : p.max_pages * kSlotTok; }
        s_len[b] = len;
    }
    if (tid == 0) {
        for (int s = 0; s < kKVStages; ++s) {
            ptx::mbar_init(&ctrl->k_full[s], 2); ptx::mbar_init(&ctrl->k_empty[s], 1);
            ptx::mbar_init(&ctrl->v_full[s], 2); ptx::mbar_init(&ctrl->v_empty[s], 1);
        }
        for (int s = 0; s < 2; ++s) { ptx::mbar_init(&ctrl->s_full[s], 1); ptx::mbar_init(&ctrl->s_free[s], 4); }
        ptx::mbar_init(&ctrl->q_full, 4);
        ptx::mbar_init(&ctrl->p_full, 4);
        ptx::mbar_init(&ctrl->pv_done, 1);
        ctrl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tm_k);
        ptx::prefetch_tmap(&tm_v);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&ctrl->tmem_base, 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
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
    const uint32_t tmem_base = ctrl->tmem_base;
    const long long tiles_per_layer = (long long)p.Hkv * cumT[p.B];
    const long long total_tiles = tiles_per_layer * p.L;
    // never more groups than tiles, so that every group's range is non-empty and boundaries are distinct
    const int n_groups = (int)min((long long)p.n_groups, total_tiles);
    const long long x_begin = group < n_groups ? total_tiles * group / n_groups : 0;
    const long long x_end = group < n_groups ? total_tiles * (group + 1) / n_groups : 0;

    if (warp == 0) {
        // =========================================================================== producer
        int ks = 0, vs = 0;
        uint32_t kph = 0, vph = 0;
        int issued = 0;
        bool ok = true;
        long long x = x_begin;
        while (x < x_end && ok) {
            const UnitPos u = locate(x, p, cumT, tiles_per_layer);
            const int len = s_len[u.b];
            const int pages_full = len / kSlotTok, pages_all = (len + kSlotTok - 1) / kSlotTok;
            const int slots_all = pages_all + p.tree_slots;
            const int t_last = (int)min((long long)u.tiles_in_unit, (long long)u.tile_in_unit + (x_end - x));
            const int32_t* pt = p.page_table + (size_t)u.b * p.max_pages;
            for (int t = u.tile_in_unit; t < t_last && ok; ++t, ++x) {
                bool w = true;
                if (lane == 0)
                    w = !ctrl->abort && ptx::mbar_wait(&ctrl->k_empty[ks], kph ^ 1) && ptx::mbar_wait(&ctrl->v_empty[vs], vph ^ 1);
                w = __shfl_sync(0xffffffffu, w, 0);
                if (!w) { if (lane == 0) timeout(p, ctrl, 10); ok = false; break; }
                uint8_t* dk = sK + (size_t)ks * C::kOperandBytes;
                uint8_t* dv = sV + (size_t)vs * C::kOperandBytes;
                const int sl0 = t * kTileSlots;
                const int n_slots = min(kTileSlots, slots_all - sl0);               // slots that exist in this tile
                const int n_tma = max(0, min(kTileSlots, pages_full - sl0));        // leading slots that are whole pages
                if (lane == 0) {
                    ptx::fence_proxy_async();          // earlier plain stores to these stages precede the bulk copies
                    ptx::mbar_arrive_expect_tx(&ctrl->k_full[ks], (uint32_t)(n_tma * C::kHalves * C::kSlotBoxBytes));
                    ptx::mbar_arrive_expect_tx(&ctrl->v_full[vs], (uint32_t)(n_tma * C::kHalves * C::kSlotBoxBytes));
                }
                __syncwarp();
                // one box per (slot, 64-column half, tensor), spread over the lanes
                for (int i = lane; i < n_tma * C::kHalves * 2; i += 32) {
                    const int j = i / (C::kHalves * 2), half = (i / 2) % C::kHalves, is_v = i & 1;
                    int page = pt[sl0 + j];
                    if (page < 0 || page >= p.num_pages) { dev_check(p, 400); page = 0; }
                    const int pg = u.layer * p.layer_pages + page;
                    if (is_v)
                        ptx::tma_load_5d(dv + half * kHalfBytes + j * C::kSlotBoxBytes, &tm_v, &ctrl->v_full[vs], 0, 0, half, u.g, pg);
                    else
                        ptx::tma_load_5d(dk + half * kHalfBytes + j * C::kSlotBoxBytes, &tm_k, &ctrl->k_full[ks], 0, 0, half, u.g, pg);
                }
                // ragged page and tree tokens by plain loads (rows beyond the valid count are zero)
                for (int j = n_tma; j < n_slots; ++j) {
                    const int sl = sl0 + j;
                    const __nv_bfloat16 *ksrc, *vsrc;
                    size_t row_stride;
                    int valid;
                    if (sl < pages_all) {
                        int page = pt[sl];
                        if (page < 0 || page >= p.num_pages) { if (lane == 0) dev_check(p, 401); page = 0; }
                        const size_t off = (((size_t)u.layer * p.layer_pages + page) * p.Hkv + u.g) * (size_t)(kSlotTok * D);
                        ksrc = p.k_pool + off; vsrc = p.v_pool + off;
                        row_stride = D;
                        valid = len - pages_full * kSlotTok;
                    } else {
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
                        *reinterpret_cast<uint4*>(dk + tile_off(j * kSlotTok + tr, cc)) = kvv;
                        *reinterpret_cast<uint4*>(dv + tile_off(j * kSlotTok + tr, cc)) = vvv;
                    }
                }
                ptx::fence_proxy_async();              // plain stores above are read by the tensor core (async proxy)
                __syncwarp();
                if (lane == 0) { ptx::mbar_arrive(&ctrl->k_full[ks]); ptx::mbar_arrive(&ctrl->v_full[vs]); }
                if (++ks == kKVStages) { ks = 0; kph ^= 1; }
                if (++vs == kKVStages) { vs = 0; vph ^= 1; }
                ++issued;
            }
        }
        if (!ok && lane == 0) {
            // let copies already in flight land before the CTA's shared memory goes away
            const int back = issued < kKVStages ? issued : kKVStages;
            for (int j = 0; j < back; ++j) {
                if (--ks < 0) { ks = kKVStages - 1; kph ^= 1; }
                if (--vs < 0) { vs = kKVStages - 1; vph ^= 1; }
                ptx::mbar_wait(&ctrl->k_full[ks], kph, 100000000ull);
                ptx::mbar_wait(&ctrl->v_full[vs], vph, 100000000ull);
            }
        }
    } else if (warp == 1) {
        // =========================================================================== UMMA issuer
        if (lane == 0) {
            const uint32_t q_addr = ptx::smem_u32(sQ), p_addr = ptx::smem_u32(sP);
            const uint32_t k_addr = ptx::smem_u32(sK), v_addr = ptx::smem_u32(sV);
            const uint32_t idesc_pv = ptx::umma_idesc_bf16(kRows, D) | (1u << 16);      // B operand MN-major
            int ks = 0, vs = 0, sb = 0;
            uint32_t kph = 0, vph = 0, sph = 0, qph = 0, pph = 0;
            bool ok = true;
            long long x = x_begin;

            auto issue_qk = [&](int n_slots) -> bool {
                if (ctrl->abort || !ptx::mbar_wait(&ctrl->k_full[ks], kph) || !ptx::mbar_wait(&ctrl->s_free[sb], sph ^ 1)) return false;
                ptx::tc_fence_after();
                const uint32_t idesc = ptx::umma_idesc_bf16(kRows, n_slots * kSlotTok);
                const uint32_t kb = k_addr + (uint32_t)(ks * C::kOperandBytes);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (uint32_t)((kk >> 2) * kHalfBytes + (kk & 3) * 32);
                    ptx::umma_f16(tmem_base + (uint32_t)(sb * kTileTok), ptx::umma_desc_k_sw128(q_addr + off),
                                  ptx::umma_desc_k_sw128(kb + off), idesc, kk != 0);
                }
                ptx::umma_commit(&ctrl->k_empty[ks]);
                ptx::umma_commit(&ctrl->s_full[sb]);
                if (++ks == kKVStages) { ks = 0; kph ^= 1; }
                if (++sb == 2) { sb = 0; sph ^= 1; }
                return true;
            };

            while (x < x_end && ok) {
                const UnitPos u = locate(x, p, cumT, tiles_per_layer);
                const int len = s_len[u.b];
                const int slots_all = (len + kSlotTok - 1) / kSlotTok + p.tree_slots;
                const int t_last = (int)min((long long)u.tiles_in_unit, (long long)u.tile_in_unit + (x_end - x));
                const int t_first = u.tile_in_unit;
                if (ctrl->abort || !ptx::mbar_wait(&ctrl->q_full, qph)) { timeout(p, ctrl, 20); ok = false; break; }
                qph ^= 1;
                if (!issue_qk(min(kTileSlots, slots_all - t_first * kTileSlots))) { timeout(p, ctrl, 21); ok = false; break; }
                for (int t = t_first; t < t_last; ++t, ++x) {
                    if (t + 1 < t_last)
                        if (!issue_qk(min(kTileSlots, slots_all - (t + 1) * kTileSlots))) { timeout(p, ctrl, 22); ok = false; break; }
                    if (ctrl->abort || !ptx::mbar_wait(&ctrl->p_full, pph) || !ptx::mbar_wait(&ctrl->v_full[vs], vph)) {
                        timeout(p, ctrl, 23); ok = false; break;
                    }
                    pph ^= 1;
                    ptx::tc_fence_after();
                    const int n_slots = min(kTileSlots, slots_all - t * kTileSlots);
                    const uint32_t vb = v_addr + (uint32_t)(vs * C::kOperandBytes);
                    for (int k = 0; k < n_slots; ++k) {
                        const uint32_t a_off = (uint32_t)((k >> 2) * kHalfBytes + (k & 3) * 32);
                        ptx::umma_f16(tmem_base + 2 * kTileTok, ptx::umma_desc_k_sw128(p_addr + a_off),
                                      umma_desc_mn_sw128(vb + (uint32_t)(k * kSlotTok * 128)), idesc_pv, (t != t_first) || (k != 0));
                    }
                    ptx::umma_commit(&ctrl->v_empty[vs]);
                    ptx::umma_commit(&ctrl->pv_done);
                    if (++vs == kKVStages) { vs = 0; vph ^= 1; }
                }
            }
        }
    } else {
        // =========================================================================== softmax / epilogue
        const int w4 = warp & 3;                                   // TMEM lane quarter of this warp
        const int row_in_blk = w4 * 32 + lane;
        const int rb_row0 = rb * p.rows_per_rb;
        const int rb_rows = min(p.rows_per_rb, p.rows - rb_row0);
        const bool row_ok = row_in_blk < rb_rows;
        const bool warp_has_rows = w4 * 32 < rb_rows;
        const int r_abs = rb_row0 + row_in_blk;                    // row within the unit: node * G + local head
        const int node = row_ok ? r_abs / p.G : 0, hl = row_ok ? r_abs % p.G : 0;
        const unsigned long long anc0 = tree.anc[node][0], anc1 = tree.anc[node][1];
        const uint32_t lane_base = tmem_base + ((uint32_t)(w4 * 32) << 16);
        const uint32_t o_taddr = lane_base + 2 * kTileTok;
        int sb = 0;
        uint32_t sph = 0, dph = 0;
        bool ok = true;
        long long x = x_begin;
        while (x < x_end && ok) {
            const UnitPos u = locate(x, p, cumT, tiles_per_layer);
            const int len = s_len[u.b];
            const int pages_full = len / kSlotTok, pages_all = (len + kSlotTok - 1) / kSlotTok;
            const int slots_all = pages_all + p.tree_slots;
            const int t_first = u.tile_in_unit;
            const int t_last = (int)min((long long)u.tiles_in_unit, (long long)t_first + (x_end - x));
            const bool whole_unit = (t_first == 0 && t_last == u.tiles_in_unit);

            // ---- Q rows of this unit into the swizzled A-operand tile (rows that do not exist are zero)
            {
                const __nv_bfloat16* qrow = p.q + ((((size_t)u.layer * p.B + u.b) * p.n + node) * (size_t)p.Hq + u.g * p.G + hl) * D;
#pragma unroll
                for (int cc = 0; cc < D / 8; ++cc) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (row_ok) v = *reinterpret_cast<const uint4*>(qrow + cc * 8);
                    *reinterpret_cast<uint4*>(sQ + tile_off(row_in_blk, cc)) = v;
                }
                ptx::fence_proxy_async();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&ctrl->q_full);
            }
            float m_used = -INFINITY, l_run = 0.f;

            for (int t = t_first; t < t_last; ++t, ++x) {
                if (ctrl->abort || !ptx::mbar_wait(&ctrl->s_full[sb], sph)) { timeout(p, ctrl, 30); ok = false; break; }
                ptx::tc_fence_after();
                float s[kTileTok];
                if (warp_has_rows) {
#pragma unroll
                    for (int c4 = 0; c4 < kTileTok / 32; ++c4) {
                        uint32_t r[32];
                        ptx::tmem_ld_32x32b_x32(lane_base + (uint32_t)(sb * kTileTok + c4 * 32), r);
#pragma unroll
                        for (int j = 0; j < 32; ++j) s[c4 * 32 + j] = __uint_as_float(r[j]);
                    }
                    ptx::tmem_ld_wait();
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&ctrl->s_free[sb]);
                if (++sb == 2) { sb = 0; sph ^= 1; }

                float mx = -INFINITY;
                if (warp_has_rows) {
                    // mask: only tiles that hold a ragged page, tree tokens or missing slots need it
                    const int sl0 = t * kTileSlots;
                    if (sl0 + kTileSlots > pages_full) {
#pragma unroll
                        for (int j = 0; j < kTileSlots; ++j) {
                            const int sl = sl0 + j;
                            if (sl < pages_full) continue;
#pragma unroll
                            for (int tr = 0; tr < kSlotTok; ++tr) {
                                bool vis;
                                if (sl < pages_all) vis = (sl * kSlotTok + tr) < len;
                                else if (sl < slots_all) {
                                    const int jt = (sl - pages_all) * kSlotTok + tr;
                                    vis = jt < p.n && (((jt < 64) ? (anc0 >> jt) : (anc1 >> (jt - 64))) & 1ull);
                                } else vis = false;
                                if (!vis) s[j * kSlotTok + tr] = -INFINITY;
                            }
                        }
                    }
#pragma unroll
                    for (int j = 0; j < kTileTok; ++j) mx = fmaxf(mx, s[j]);
                }
                // the previous tile's P V must be complete before P is overwritten or O is touched
                if (t != t_first) {
                    if (ctrl->abort || !ptx::mbar_wait(&ctrl->pv_done, dph)) { timeout(p, ctrl, 31); ok = false; break; }
                    dph ^= 1;
                    ptx::tc_fence_after();
                }
                if (warp_has_rows) {
                    // offset in use: moved only at the first tile or when the row maximum outgrew it by 2^8
                    const bool move = (t == t_first) || ((mx - m_used) * p.scale_log2e > kRescaleLog2) ||
                                      (m_used == -INFINITY && mx > -INFINITY);
                    const float m_next = move ? fmaxf(mx, m_used) : m_used;
                    if (t != t_first && __any_sync(0xffffffffu, move)) {
                        const float alpha = (m_used == -INFINITY) ? ((m_next == -INFINITY) ? 1.f : 0.f)
                                                                  : exp2f((m_used - m_next) * p.scale_log2e);
#pragma unroll
                        for (int c4 = 0; c4 < D / 32; ++c4) {
                            uint32_t r[32];
                            ptx::tmem_ld_32x32b_x32(o_taddr + (uint32_t)(c4 * 32), r);
                            ptx::tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * alpha);
                            tmem_st_32x32b_x32(o_taddr + (uint32_t)(c4 * 32), r);
                        }
                        tmem_st_wait();
                        l_run *= alpha;
                    }
                    m_used = m_next;
                    const float off = (m_used == -INFINITY) ? 0.f : m_used * p.scale_log2e;
                    float sum = 0.f;
#pragma unroll
                    for (int c8 = 0; c8 < kTileTok / 8; ++c8) {
                        float e[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) { e[j] = exp2f(fmaf(s[c8 * 8 + j], p.scale_log2e, -off)); sum += e[j]; }
                        uint4 v;
                        v.x = pack_bf16(e[0], e[1]); v.y = pack_bf16(e[2], e[3]); v.z = pack_bf16(e[4], e[5]); v.w = pack_bf16(e[6], e[7]);
                        *reinterpret_cast<uint4*>(sP + tile_off(row_in_blk, c8)) = v;
                    }
                    l_run += sum;
                }
                ptx::fence_proxy_async();
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&ctrl->p_full);
            }
            if (!ok) break;
            // ---- end of this CTA's part of the unit: read O once the last P V is complete
            if (ctrl->abort || !ptx::mbar_wait(&ctrl->pv_done, dph)) { timeout(p, ctrl, 32); ok = false; break; }
            dph ^= 1;
            ptx::tc_fence_after();
            if (!warp_has_rows) continue;

            __nv_bfloat16* orow = p.out + ((((size_t)u.layer * p.B + u.b) * p.n + node) * (size_t)p.Hq + u.g * p.G + hl) * D;
            float* lse_ptr = p.lse_out ? p.lse_out + (((size_t)u.layer * p.B + u.b) * p.Hq + u.g * p.G + hl) * p.n + node : nullptr;

            if (whole_unit) {
                const float inv = 1.f / l_run;
#pragma unroll
                for (int c4 = 0; c4 < D / 32; ++c4) {
                    uint32_t r[32];
                    ptx::tmem_ld_32x32b_x32(o_taddr + (uint32_t)(c4 * 32), r);
                    ptx::tmem_ld_wait();
                    if (row_ok) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint4 v;
                            v.x = pack_bf16(__uint_as_float(r[j * 8 + 0]) * inv, __uint_as_float(r[j * 8 + 1]) * inv);
                            v.y = pack_bf16(__uint_as_float(r[j * 8 + 2]) * inv, __uint_as_float(r[j * 8 + 3]) * inv);
                            v.z = pack_bf16(__uint_as_float(r[j * 8 + 4]) * inv, __uint_as_float(r[j * 8 + 5]) * inv);
                            v.w = pack_bf16(__uint_as_float(r[j * 8 + 6]) * inv, __uint_as_float(r[j * 8 + 7]) * inv);
                            *reinterpret_cast<uint4*>(orow + c4 * 32 + j * 8) = v;
                        }
                    }
                }
                if (lse_ptr && row_ok) *lse_ptr = m_used * p.scale + logf(l_run);
                ptx::tc_fence_before();
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
            const int slot = (t_first > 0) ? 0 : 1;      // a unit that began before this CTA's range uses slot 0
            constexpr int kRowW = D + 2;
            float* my = p.partial + (((size_t)blockIdx.x * 2 + slot) * kRows + row_in_blk) * kRowW;
#pragma unroll
            for (int c4 = 0; c4 < D / 32; ++c4) {
                uint32_t r[32];
                ptx::tmem_ld_32x32b_x32(o_taddr + (uint32_t)(c4 * 32), r);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    *reinterpret_cast<float2*>(my + c4 * 32 + j * 2) = make_float2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
            }
            *reinterpret_cast<float2*>(my + D) = make_float2(m_used, l_run);
            ptx::tc_fence_before();
            __threadfence();
            __syncwarp();
            const size_t unit_idx = ((size_t)u.layer * p.B + u.b) * p.Hkv + u.g;
            int* tk = p.ticket + (unit_idx * p.n_rb + rb) * kMergeWarps + w4;
            int arrived = 0;
            if (lane == 0) arrived = atomicAdd(tk, 1);
            arrived = __shfl_sync(0xffffffffu, arrived, 0);
            if (arrived != parts - 1) continue;
            __threadfence();
            if (lane == 0) *tk = 0;                              // ready for the next launch
            if (!row_ok) continue;
            // merge in group order
            float M = -INFINITY;
            for (int gsrc = ga; gsrc <= gb; ++gsrc) {
                const int sslot = (per * gsrc / n_groups > u.unit_first_tile) ? 0 : 1;
                const float* src = p.partial + (((size_t)(gsrc * p.n_rb + rb) * 2 + sslot) * kRows + row_in_blk) * kRowW;
                M = fmaxf(M, __ldcg(src + D));
            }
            float Lsum = 0.f;
            float acc[D];
#pragma unroll
            for (int j = 0; j < D; ++j) acc[j] = 0.f;
            for (int gsrc = ga; gsrc <= gb; ++gsrc) {
                const int sslot = (per * gsrc / n_groups > u.unit_first_tile) ? 0 : 1;
                const float* src = p.partial + (((size_t)(gsrc * p.n_rb + rb) * 2 + sslot) * kRows + row_in_blk) * kRowW;
                const float2 ml = __ldcg(reinterpret_cast<const float2*>(src + D));
                const float wgt = (ml.x == -INFINITY) ? 0.f : exp2f((ml.x - M) * p.scale_log2e);
                Lsum += wgt * ml.y;
#pragma unroll
                for (int j = 0; j < D / 2; ++j) {
                    const float2 v = __ldcg(reinterpret_cast<const float2*>(src + 2 * j));
                    acc[2 * j] += wgt * v.x; acc[2 * j + 1] += wgt * v.y;
                }
            }
            const float inv = 1.f / Lsum;
#pragma unroll
            for (int j = 0; j < D / 8; ++j) {
                uint4 v;
                v.x = pack_bf16(acc[j * 8 + 0] * inv, acc[j * 8 + 1] * inv);
                v.y = pack_bf16(acc[j * 8 + 2] * inv, acc[j * 8 + 3] * inv);
                v.z = pack_bf16(acc[j * 8 + 4] * inv, acc[j * 8 + 5] * inv);
                v.w = pack_bf16(acc[j * 8 + 6] * inv, acc[j * 8 + 7] * inv);
                *reinterpret_cast<uint4*>(orow + j * 8) = v;
            }
            if (lse_ptr) *lse_ptr = M * p.scale + logf(Lsum);
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, 512);
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
    p.n_rb = (p.rows + kRows - 1) / kRows;
    p.rows_per_rb = (p.rows + p.n_rb - 1) / p.n_rb;
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
    if ((size_t)p.L * p.B * Hkv * p.n_rb * kMergeWarps > ticket_ints) return MIRROR_ERR_WORKSPACE;
    if (p.B > kMaxBatch) return MIRROR_ERR_SHAPE;

    AttnTree at;
    memcpy(at.anc, ti.anc, sizeof at.anc);

    CUtensorMap tm_k, tm_v;
    {
        // pool viewed as (64 columns, 16 tokens, D/64 halves, Hkv heads, layers*pages); one box = one half of one page
        const uint64_t total_pages = (uint64_t)(p.L - 1) * p.layer_pages + p.num_pages;
        const uint64_t dims[5] = {64, (uint64_t)kSlotTok, (uint64_t)(D / 64), (uint64_t)Hkv, total_pages};
        const uint64_t strides[4] = {(uint64_t)D * 2, 128, (uint64_t)kSlotTok * D * 2, (uint64_t)page_elems * 2};
        const uint32_t box[5] = {64, (uint32_t)kSlotTok, 1, 1, 1};
        mirror_status st = mirror_make_tmap(ctx, &tm_k, kv->k_pool, 5, dims, strides, box);
        if (st != MIRROR_OK) return st;
        st = mirror_make_tmap(ctx, &tm_v, kv->v_pool, 5, dims, strides, box);
        if (st != MIRROR_OK) return st;
    }
    const int grid = p.n_groups * p.n_rb;
    if (D == 128) {
        MIRROR_CUDA_OK(cudaFuncSetAttribute(attn_verify_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<128>::kSmemBytes));
        attn_verify_kernel<128><<<grid, kThreads, Cfg<128>::kSmemBytes, stream>>>(tm_k, tm_v, at, p);
    } else {
        MIRROR_CUDA_OK(cudaFuncSetAttribute(attn_verify_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<64>::kSmemBytes));
        attn_verify_kernel<64><<<grid, kThreads, Cfg<64>::kSmemBytes, stream>>>(tm_k, tm_v, at, p);
    }
    ctx->launches += 1;
    MIRROR_CUDA_OK(cudaGetLastError());
    return MIRROR_OK;
}
