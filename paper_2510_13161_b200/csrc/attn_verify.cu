// Branch-tree attention of the verify step: every tree node (kappa x gamma draft tokens + the root)
// attends to the paged KV cache of the verified prefix and to the tree's own K/V under the
// branch-causal mask (node i sees tree token j iff j is i or an ancestor of i), for all layers.
//
// Work decomposition.  A "unit" is (layer, request, KV head): all G = Hq/Hkv query heads of all n tree
// nodes (G*n rows) share that head's K/V stream, so one CTA owning the unit's rows reads each K/V byte
// once from HBM and reuses it from shared memory for every row (the GQA / tree sharing).  A unit's keys
// are cut into 16-token slots (one KV page, or 16 tree tokens); four slots form a 64-token tile and a ring stage.  A
// slot lands in shared memory as [token / 8][64-column half][token % 8][128 B] (one 5-D TMA box per page), so that the
// 8-token groups of a half are evenly spaced across slots and stages: two consecutive stages are one K-major UMMA
// operand of up to 128 tokens in token order, and each slot is one MN-major 16-token P V step.  The tiles of all
// units form one sequence that is split evenly over persistent CTAs (one per SM), so a unit may be cut
// across CTAs; each CTA then leaves a partial (max, sum, accumulator) and a small second kernel merges the parts
// of every cut unit in a fixed order (no counters, fences or atomics: no CTA ever waits for, or signals, another).
// More than 128 rows per unit are handled by row blocks: a group of CTAs walks the same tiles at the
// same time, each with its own rows, so the second read of a tile is served by L2.
//
// Per CTA (12 warps):
//   warp 0, 11  stage K and V into two rings of 4-slot stages (4 or 6 deep: whatever the Q buffers leave): one TMA box
//               per page and tensor, 128-byte swizzle; ragged page and tree tokens by 16-byte asynchronous copies
//               with zero fill
//   warp 1      owns TMEM and issues S = Q K^T tile by tile (tcgen05.mma, M=128 rows, N up to 64 tokens, d/16
//               instructions) into one of four S buffers, as far ahead as rings and buffers allow; Q is
//               double-buffered, so it runs on into the next unit while the softmax warps finish this one
//   warp 2      issues O += P V (P as the A operand from tensor memory, V as an MN-major operand from shared memory)
//   warps 3..10 softmax, two groups of four warps on alternate tiles, one thread per row (TMEM lane): ONE pass over the
//               row's 64 scores: P = exp2(s*c - offset) against the offset in use, written as bf16 over the first half
//               of the same S buffer (the buffer is released by the P V that reads it); no shuffles, no shared memory,
//               and no row maximum on the way: the offset is set by the row's first tile and moves only when a tile's
//               SUM of P outgrows 2^14 (that tile is then redone; the stale offset is carried exactly through the sum
//               and the division); each group keeps its own accumulator O in TMEM and the two are merged like
//               split-KV partials; they also stage the next unit's Q a unit ahead
// Every ring index and mbarrier parity is a function of one per-CTA tile counter, identical in all roles.
// Every mbarrier wait is bounded; on expiry the kernel records MIRROR_DEV_TIMEOUT and unwinds.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <type_traits>

#include "mirror_internal.h"

namespace {

constexpr int kSoftmaxWarps = 8;
constexpr int kThreads = 32 * (4 + kSoftmaxWarps);   // K producer, Q K^T issuer, P V issuer, softmax pairs, V producer
constexpr int kVProducerWarp = 3 + kSoftmaxWarps;
constexpr int kSlotTok = 16;
constexpr int kTileSlots = 4;
constexpr int kTileTok = kSlotTok * kTileSlots;     // 64
constexpr int kRows = 128;                          // UMMA M: rows per row block
constexpr int kMaxBatch = 1024;
constexpr int kMaxStages = 8;                       // ring depths are template parameters (even: tiles are staged in pairs)
constexpr int kSBufs = 4;                           // S buffers in TMEM (power of two)
// A row's offset puts the maximum of the tile that set it at 2^bias and moves when a tile's sum of P passes the limit
// (no single P is beyond the limit then).  bf16 P: 2^0 and 2^14.  e4m3 P: 2^2 and 448, the largest e4m3 value (a tile
// of 64 equal scores sums to 256); weights below 2^-12 of the maximum that set the offset round to zero.
template <bool F8> struct POffset {
    static constexpr float kBias = F8 ? 2.0f : 0.0f;
    static constexpr float kSumLimit = F8 ? 448.0f : 16384.0f;
};
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kTmemCols = 512;                      // S0..S3 (64 columns each; P overwrites the first 32 of its S) | O of group 0 | O of group 1
constexpr int kTmemO = kSBufs * kTileTok;

struct AttnTree {
    unsigned long long anc[MIRROR_MAX_NODES][2];
};

struct AttnParams {
    int L, B, n, Hq, Hkv, G;
    int rows, n_rb, rows_per_rb;          // rows per unit, row blocks, rows per block
    int n_groups;                         // CTA groups (grid = n_groups * n_rb)
    int snap_cap;                         // boundaries move to a unit boundary that is at most this many tiles away
    int whole_units;                      // 1: prefer a group count that divides equal-length units (no cuts)
    int max_pages, num_pages, layer_pages;
    int q_half_bytes;                     // one 64-column half of a Q buffer: rows rounded up to 8, 128 B each
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
    float* partial;                       // [grid][2][D+4][128]
    int* status;
    // e4m3 cache: pools, k_new and v_new hold e4m3 codes (one byte per element); a code times its (layer, KV head)
    // scale is the value.  Q stays bf16 in memory; its operand is e4m3(q / q_scale), rounded when it is staged.
    const float* k_scale;                 // [L, Hkv]
    const float* v_scale;                 // [L, Hkv]
    float q_scale;
    long long wait_limit;                 // SM cycles after which a wait gives up
    int stall_after;                      // test aid: the K producer stops after this many stages (-1: never)
};

struct UnitPos {                          // where a global tile index falls
    int layer, b, g;
    int tile_in_unit, tiles_in_unit;
    long long unit_first_tile;            // global index of the unit's first tile
};

struct Ctrl {
    uint64_t k_full[kMaxStages], k_empty[kMaxStages];   // K ring: refilled as soon as Q K^T has read a stage
    uint64_t v_full[kMaxStages], v_empty[kMaxStages];   // V ring: refilled once P V has read a stage
    uint64_t s_full[kSBufs], s_free[kSBufs];
    uint64_t p_full[kSBufs], pv_done[2];
    uint64_t q_full[2];
    uint64_t pair[4];                                   // softmax warp pairs' exchange
    uint64_t o_free;                                    // accumulators read out at the end of a unit's part
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

// A bounded wait that looks at the CTA's abort flag only when the barrier is not complete yet (the common case is one
// try_wait), and between parks while it waits.
__device__ __forceinline__ bool wait_bar(Ctrl* c, uint64_t* bar, uint32_t parity, long long limit_cycles) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (c->abort) return false;
        if (ptx::mbar_try_wait_park(bar, parity, MIRROR_PARK_NS)) return true;
        if (clock64() - t0 > limit_cycles) return false;
    }
}

// Two barriers at once: both polls are issued before either result is looked at.
__device__ __forceinline__ bool wait_bar2(Ctrl* c, uint64_t* bar_a, uint32_t par_a, uint64_t* bar_b, uint32_t par_b, long long limit_cycles) {
    const bool a = ptx::mbar_try_wait(bar_a, par_a), b = ptx::mbar_try_wait(bar_b, par_b);
    if (a && b) return true;
    return (a || wait_bar(c, bar_a, par_a, limit_cycles)) && (b || wait_bar(c, bar_b, par_b, limit_cycles));
}

__device__ __noinline__ UnitPos locate(long long x, const AttnParams& p, const int* cumT, long long tiles_per_layer) {
    UnitPos u;
    // (the tile count fits 31 bits: checked in the prologue; 32-bit divisions are several times cheaper)
    u.layer = (int)((uint32_t)x / (uint32_t)tiles_per_layer);
    const long long rem = x - (long long)u.layer * tiles_per_layer;
    int b = 0;
    while (b + 1 < p.B && (long long)p.Hkv * cumT[b + 1] <= rem) ++b;
    const int Tb = cumT[b + 1] - cumT[b];
    const long long r2 = rem - (long long)p.Hkv * cumT[b];
    u.b = b;
    u.g = (int)((uint32_t)r2 / (uint32_t)Tb);
    u.tile_in_unit = (int)(r2 - (long long)u.g * Tb);
    u.tiles_in_unit = Tb;
    u.unit_first_tile = x - u.tile_in_unit;
    return u;
}

// P = exp2(x) for two fp32 arguments: the pair rounded to bf16 (element `lo` in the low half, as the tensor core reads P);
// the fp32 values are added to two running sums.
__device__ __forceinline__ uint32_t exp2_pair(float lo, float hi, float& sum_lo, float& sum_hi) {
    const float e0 = ptx::ex2_approx(lo), e1 = ptx::ex2_approx(hi);
    sum_lo += e0;
    sum_hi += e1;
    uint32_t pk;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(e1), "f"(e0));
    return pk;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float m;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(m) : "f"(a), "f"(b), "f"(c));
    return m;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Four fp32 values as e4m3 codes in one word (element 0 in the lowest byte, as the tensor core reads an 8-bit operand);
// values beyond +-448 saturate.
__device__ __forceinline__ uint32_t pack_e4m3x4(float a, float b, float c, float d) {
    uint32_t r;
    asm("{\n\t.reg .b16 lo, hi;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
        "mov.b32 %0, {lo, hi};\n\t}"
        : "=r"(r) : "f"(a), "f"(b), "f"(c), "f"(d));
    return r;
}
// tcgen05.mma with both operands in shared memory (descriptor halves) or A in tensor memory; F8 selects e4m3 inputs.
template <bool F8>
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                        uint32_t idesc, uint32_t accumulate) {
    if constexpr (F8) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
            "mov.b64 da, {%1, %2};\n\t"
            "mov.b64 db, {%3, %4};\n\t"
            "setp.ne.b32 p, %6, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %5, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
            : "memory");
    } else {
        ptx::umma_f16_lohi(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc, accumulate);
    }
}
template <bool F8>
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                        uint32_t accumulate) {
    if constexpr (F8) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
            "mov.b64 db, {%2, %3};\n\t"
            "setp.ne.b32 p, %5, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], db, %4, p;\n\t}"
            ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
            : "memory");
    } else {
        ptx::umma_f16_tmem_a(d_tmem, a_tmem, b_lo, b_hi, idesc, accumulate);
    }
}
// Instruction descriptor: e4m3 x e4m3 -> fp32 (format codes 0), tile M x N.
__device__ __forceinline__ uint32_t umma_idesc_e4m3(int M, int N) {
    return (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Shared-memory operand tiles are [64-column half][row][128 B] with the 128-byte swizzle: the 16-byte chunk
// index is XORed with (row % 8).  A half of Q or P holds 128 rows (16 KB), a half of a K/V stage 64 tokens (8 KB).
constexpr int kStageSlots = 4;                      // slots per ring stage
// A K/V slot (16 tokens of one head) is [token / 8][64-column half][token % 8][128 B]: the 8-token groups of one half
// are 1024 * (d / 64) bytes apart, uniformly across the slots of a ring, which is the 8-row-group stride (SBO) of the
// K-major Q K^T operand over up to 128 tokens and, with the halves 1024 B apart (LBO), the MN-major P V operand.
// (An e4m3 row of 128 elements is a single 128-byte half.)
template <int HALVES>
__device__ __forceinline__ uint32_t kv_slot_off(int tok, int chunk) {                 // chunk: 16-byte column chunk
    return (uint32_t)((tok >> 3) * HALVES * 1024 + (chunk >> 3) * 1024 + (tok & 7) * 128 + (((chunk & 7) ^ (tok & 7)) << 4));
}
__device__ __forceinline__ uint32_t tile_off(int row, int chunk, int half_bytes) {   // chunk: 16-byte column chunk
    return (uint32_t)((chunk >> 3) * half_bytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
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
__device__ __forceinline__ void tmem_st_32x32b_x16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }


template <int D, bool F8>
struct Cfg {
    static_assert(!F8 || D == 128, "an e4m3 row must fill a 128-byte swizzle row");
    static constexpr int kElemBytes = F8 ? 1 : 2;
    static constexpr int kRowBytes = D * kElemBytes;               // one token's K (or V) row of one head
    static constexpr int kHalves = kRowBytes / 128;
    static constexpr int kSlotBytes = kHalves * kSlotTok * 128;    // one slot of K or V (see kv_slot_off) = one TMA box
    static constexpr int kGroupStride = kHalves * 1024;            // between the 8-token groups of one half
    static constexpr int kStageBytes = kStageSlots * kSlotBytes;   // one K (or V) stage: 4 slots; stages are contiguous
    static constexpr size_t kSmemFixed = 512 /*ctrl*/ + 2 * 2 * kRows * 4 /*pair exchange*/ + (2 * kMaxBatch + 2) * 4 + 1024 /*align*/;
    // Shared memory: two Q buffers sized by the rows a CTA really has (the UMMA reads 128 rows per half and
    // runs on into whatever follows; those rows only reach TMEM lanes nobody reads), then the K and V rings.
    // What the rings can hold in flight bounds the bandwidth one SM can pull at HBM latency, so they get
    // every byte the Q buffers leave.
    static size_t smem_bytes(int q_half_bytes, int ks, int vs) {
        return 2 * (size_t)kHalves * q_half_bytes + (size_t)(ks + vs) * kStageBytes + kSmemFixed;
    }
};

// Visibility of 32 score columns (the 16 tokens of slots sl0 and sl0 + 1) for a row whose visible tree tokens are the
// bits of (anc0, anc1).  Kept out of line and rolled: it runs for a unit's last tiles only.
__device__ __noinline__ uint32_t chunk_mask(int sl0, int pages_full, int pages_all, int slots_all, int len,
                                            unsigned long long anc0, unsigned long long anc1) {
    uint32_t cm = 0;
#pragma unroll 1
    for (int jj = 0; jj < 2; ++jj) {
        const int sl = sl0 + jj;
        uint32_t bits = 0;
        if (sl < pages_full) {
            bits = 0xffffu;
        } else if (sl < pages_all) {
            bits = (1u << (len - sl * kSlotTok)) - 1u;                              // ragged page: 1..15 valid tokens
        } else if (sl < slots_all) {
            const int ts = sl - pages_all;                                          // tree tokens 16*ts .. 16*ts+15
            bits = (uint32_t)(((ts < 4) ? anc0 : anc1) >> ((ts & 3) * 16)) & 0xffffu;   // ancestors-or-self (all < n)
        }
        cm |= bits << (jj * 16);
    }
    return cm;
}

// A segment: the part of one unit that this CTA processes.
struct Segment {
    UnitPos u;
    int t_first, t_last;                  // tiles [t_first, t_last) of the unit
    int len, pages_full, pages_all, slots_all;
};
__device__ __noinline__ Segment make_segment(long long x, long long x_end, const AttnParams& p, const int* cumT,
                                                const int* s_len, long long tiles_per_layer) {
    Segment s;
    s.u = locate(x, p, cumT, tiles_per_layer);
    s.t_first = s.u.tile_in_unit;
    s.t_last = (int)min((long long)s.u.tiles_in_unit, (long long)s.t_first + (x_end - x));
    s.len = s_len[s.u.b];
    s.pages_full = s.len / kSlotTok;
    s.pages_all = (s.len + kSlotTok - 1) / kSlotTok;
    s.slots_all = s.pages_all + p.tree_slots;
    return s;
}

// How the tile sequence is cut into one range per CTA group.
// Group count that gives every group the same number of whole units, if one exists within 15% of n_groups; else 0.
// (Host and device: the host uses it to tell whether a launch can cut a unit at all.)
__host__ __device__ inline int whole_unit_groups(int n_groups, long long units) {
    for (int g = n_groups; g >= 1 && g * 100 >= n_groups * 85; --g)
        if (units % g == 0) return g;
    return 0;
}

struct Partition {
    long long tiles_per_layer, total_tiles, total_pairs, snap_tol;
    int n_groups;
};
__device__ __forceinline__ Partition make_partition(const AttnParams& p, const int* cumT) {
    Partition q;
    q.tiles_per_layer = (long long)p.Hkv * cumT[p.B];
    q.total_tiles = q.tiles_per_layer * p.L;
    // CTA groups own whole pairs of tiles; never more groups than pairs, so that every group's range is non-empty
    q.total_pairs = q.total_tiles / 2;
    q.n_groups = (int)min((long long)p.n_groups, q.total_pairs);
    // Units of equal length (every request has the same number of tiles): a group count that divides the units, if one
    // exists within 15% of the CTA groups there are, gives every group the same number of WHOLE units: no unit is cut,
    // nothing is left to merge and all groups end together, which is worth more than the few SMs left idle
    // (384 units on 148 SMs: 128 groups of 3 units, attention 111 -> 105 us).
    bool equal_units = true;
    for (int b = 1; b < p.B; ++b) equal_units &= (cumT[b + 1] - cumT[b]) == cumT[1];
    if (p.whole_units && equal_units && q.n_groups == p.n_groups) {
        const int g = whole_unit_groups(p.n_groups, (long long)p.L * p.B * p.Hkv);
        if (g > 0) q.n_groups = g;
    }
    // A boundary that falls within snap_tol tiles (a cut costs about as much as a few tiles) of a unit boundary
    // moves there: both neighbours then hold whole units and no partial has to be left and merged.  snap_tol is
    // at most a quarter of the smallest even share, so boundaries stay strictly increasing.
    q.snap_tol = q.n_groups > 0 ? min((long long)p.snap_cap, (2 * (q.total_pairs / q.n_groups)) / 4) : 0;
    return q;
}
__device__ __noinline__ long long group_begin(const Partition& q, int g, const AttnParams& p, const int* cumT) {
    if (g <= 0) return 0;
    if (g >= q.n_groups) return q.total_tiles;
    const long long e = 2 * (q.total_pairs * g / q.n_groups);
    if (q.snap_tol == 0) return e;
    const UnitPos u = locate(e, p, cumT, q.tiles_per_layer);
    const long long lo = u.unit_first_tile, hi = lo + u.tiles_in_unit;
    const long long best = (e - lo <= hi - e) ? lo : hi;
    const long long dist = best > e ? best - e : e - best;
    return dist <= q.snap_tol ? best : e;
}

template <int D, int KS, int VS, bool F8>
__global__ void __launch_bounds__(kThreads, 1)
attn_verify_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ AttnTree tree, const AttnParams p) {
    using C = Cfg<D, F8>;
    using PO = POffset<F8>;
    constexpr int KR = KS;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem;                                             // [2]: the units a CTA walks alternate
    const int q_buf_bytes = C::kHalves * p.q_half_bytes;
    uint8_t* sK = sQ + 2 * q_buf_bytes;                             // [KS]  [slot][half][16 tokens][128 B]
    uint8_t* sV = sK + KS * C::kStageBytes;                         // [VS]  [slot][half][16 tokens][128 B]
    Ctrl* ctrl = (Ctrl*)(sV + VS * C::kStageBytes);
    float* xch = (float*)((uint8_t*)ctrl + 512);                    // [2 tiles][2 halves][128 rows] pair exchange
    int* cumT = (int*)((uint8_t*)ctrl + 512 + 2 * 2 * kRows * 4);   // [B+1] tiles per request, prefix-summed
    int* s_len = cumT + (kMaxBatch + 1);                            // [B] clamped prefix lengths

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int group = blockIdx.x / p.n_rb, rb = blockIdx.x % p.n_rb;

    // ---- prologue ---------------------------------------------------------------------------------
    // (programmatic dependent launch: barriers and tensor memory are set up while the kernel ahead in the stream is
    // still running; nothing of global memory is touched before it has completed)
    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            ptx::mbar_init(&ctrl->k_full[s], 1); ptx::mbar_init(&ctrl->k_empty[s], 1);
            ptx::mbar_init(&ctrl->v_full[s], 1); ptx::mbar_init(&ctrl->v_empty[s], 1);
        }
        for (int s = 0; s < kSBufs; ++s) {
            ptx::mbar_init(&ctrl->s_full[s], 1); ptx::mbar_init(&ctrl->s_free[s], 1);     // freed by the P V that read P from it
            ptx::mbar_init(&ctrl->p_full[s], kSoftmaxWarps / 2);
        }
        for (int s = 0; s < 2; ++s) { ptx::mbar_init(&ctrl->pv_done[s], 1); ptx::mbar_init(&ctrl->q_full[s], kSoftmaxWarps); }
        for (int s = 0; s < 4; ++s) ptx::mbar_init(&ctrl->pair[s], 2);
        ptx::mbar_init(&ctrl->o_free, kSoftmaxWarps);
        ctrl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tm_k);
        ptx::prefetch_tmap(&tm_v);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&ctrl->tmem_base, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();                 // the merge kernel behind may be scheduled as soon as SMs free up
    for (int b = tid; b < p.B; b += kThreads) {
        int len = p.prefix_len[b];
        if (len < 0 || len > p.max_pages * kSlotTok) { dev_check(p, 300 + b); len = len < 0 ? 0 : p.max_pages * kSlotTok; }
        s_len[b] = len;
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        cumT[0] = 0;
        for (int b = 0; b < p.B; ++b) {
            const int slots = (s_len[b] + kSlotTok - 1) / kSlotTok + p.tree_slots;
            acc += 2 * ((slots + 2 * kStageSlots - 1) / (2 * kStageSlots));      // whole pairs of tiles
            cumT[b + 1] = acc;
        }
    }
    __syncthreads();
    const uint32_t tmem_base = ctrl->tmem_base;
    const Partition part = make_partition(p, cumT);
    const long long tiles_per_layer = part.tiles_per_layer, total_tiles = part.total_tiles;
    const int n_groups = part.n_groups;
    const bool fits = total_tiles < (1ll << 31);
    if (!fits && tid == 0) dev_check(p, 600);
    const long long x_begin = (fits && group < n_groups) ? group_begin(part, group, p, cumT) : 0;
    const long long x_end = (fits && group < n_groups) ? group_begin(part, group + 1, p, cumT) : 0;
    if (warp == 0 || warp == kVProducerWarp) {
        // =========================================================================== producers
        // warp 0 stages K, the last warp stages V: a warp issues its TMA boxes one after the other, so two
        // warps halve the time a stage takes to request
        const bool vrole = (warp == kVProducerWarp);
        uint64_t* const full = vrole ? ctrl->v_full : ctrl->k_full;
        uint64_t* const empty = vrole ? ctrl->v_empty : ctrl->k_empty;
        uint32_t it = 0;                   // tiles issued by this CTA so far (ring index and parity source)
        bool ok = true;
        long long x = x_begin;
        // one TMA box (a whole page of this tensor) per lane
        const bool has_box = lane < kStageSlots;
        const int my_slot = lane;
        while (x < x_end && ok) {
            const Segment sg = make_segment(x, x_end, p, cumT, s_len, tiles_per_layer);
            const UnitPos& u = sg.u;
            const int32_t* pt = p.page_table + (size_t)u.b * p.max_pages;
            // the page id a lane needs is fetched one tile ahead, so its latency hides behind the ring wait
            auto fetch_page = [&](int tt) -> int {
                const int sl = tt * kStageSlots + my_slot;
                return (has_box && sl < sg.pages_full) ? pt[sl] : 0;
            };
            int my_page = fetch_page(sg.t_first);
            if (sg.t_last == u.tiles_in_unit) {
                // the unit's last slots (a ragged page, the tree's own tokens) are staged by plain loads many tiles
                // from now: pull them into L2 so that those loads do not hold up the ring for an HBM round trip
                for (int j = lane; j < p.n; j += 32) {
                    const uint8_t* row = (const uint8_t*)(vrole ? p.v_new : p.k_new) + ((((size_t)u.layer * p.B + u.b) * p.n + j) * p.Hkv + u.g) * (size_t)C::kRowBytes;
                    ptx::prefetch_l2(row);
                    if (C::kRowBytes == 256) ptx::prefetch_l2(row + 128);
                }
                if (sg.pages_all > sg.pages_full) {
                    const int page = pt[sg.pages_full];
                    if (page >= 0 && page < p.num_pages && lane < kSlotTok * C::kRowBytes / 128)
                        ptx::prefetch_l2((const uint8_t*)(vrole ? p.v_pool : p.k_pool) + (((size_t)u.layer * p.layer_pages + page) * p.Hkv + u.g) * (size_t)(kSlotTok * C::kRowBytes) + lane * 128);
                }
            }
            for (int t = sg.t_first; t < sg.t_last && ok; ++t, ++x, ++it) {
                if (!vrole && p.stall_after >= 0 && (int)it >= p.stall_after) { x = x_end; break; }      // (test aid: see AttnParams)
                const int st = vrole ? (int)(it % VS) : (int)(it % KR);
                const uint32_t ph = (vrole ? it / VS : it / KR) & 1;
                const int next_page = (t + 1 < sg.t_last) ? fetch_page(t + 1) : 0;
                bool w = true;
                if (lane == 0) w = wait_bar(ctrl, &empty[st], ph ^ 1, p.wait_limit);
                w = __shfl_sync(0xffffffffu, w, 0);
                if (!w) { if (lane == 0) timeout(p, ctrl, 10); ok = false; break; }
                uint8_t* dst = (vrole ? sV : sK) + (size_t)st * C::kStageBytes;
                const int sl0 = t * kStageSlots;
                const int n_slots = max(0, min(kStageSlots, sg.slots_all - sl0));      // slots that exist in this stage
                const int n_tma = max(0, min(kStageSlots, sg.pages_full - sl0));       // leading slots that are whole pages
                // (e4m3: a P V step spans two slots, so an odd last slot gets a partner of zeros: stale bytes could be NaN codes)
                const int n_fill = F8 ? min(kStageSlots, (n_slots + 1) & ~1) : n_slots;
                if (n_tma < n_fill) {
                    // ragged page and tree tokens by asynchronous 16-byte copies (rows beyond the valid count are
                    // zero-filled), all in flight together; the loops are kept rolled: this path runs once per unit, and
                    // what it costs is mostly the instruction fetch
                    constexpr int kRowChunks = C::kRowBytes / 16;      // 16-byte chunks per token row
                    constexpr int kChunks = kSlotTok * kRowChunks;     // ... and per slot
                    constexpr int kPer = kChunks / 32;
#pragma unroll 1
                    for (int j = n_tma; j < n_fill; ++j) {
                        const int sl = sl0 + j;
                        const uint8_t* src = (const uint8_t*)p.k_pool;             // (bytes)
                        size_t row_stride = 0;
                        int valid = 0;
                        if (sl < sg.pages_all) {
                            int page = pt[sl];
                            if (page < 0 || page >= p.num_pages) { if (lane == 0) dev_check(p, 401); page = 0; }
                            src = (const uint8_t*)(vrole ? p.v_pool : p.k_pool) + (((size_t)u.layer * p.layer_pages + page) * p.Hkv + u.g) * (size_t)(kSlotTok * C::kRowBytes);
                            row_stride = C::kRowBytes;
                            valid = sg.len - sg.pages_full * kSlotTok;
                        } else if (sl < sg.slots_all) {
                            const int j0 = (sl - sg.pages_all) * kSlotTok;
                            src = (const uint8_t*)(vrole ? p.v_new : p.k_new) + ((((size_t)u.layer * p.B + u.b) * p.n + j0) * p.Hkv + u.g) * (size_t)C::kRowBytes;
                            row_stride = (size_t)p.Hkv * C::kRowBytes;
                            valid = min(kSlotTok, p.n - j0);
                        }
#pragma unroll 1
                        for (int i = 0; i < kPer; ++i) {
                            const int c = lane + i * 32, tr = c / kRowChunks, cc = c % kRowChunks;
                            const bool in = tr < valid;
                            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                                         ::"r"(ptx::smem_u32(dst + j * C::kSlotBytes + kv_slot_off<C::kHalves>(tr, cc))),
                                           "l"(in ? src + tr * row_stride + cc * 16 : (const uint8_t*)p.k_pool), "r"(in ? 16u : 0u) : "memory");
                        }
                    }
                    asm volatile("cp.async.wait_all;" ::: "memory");
                    // these copies are read by the tensor core, and later overwritten by bulk copies (async proxy)
                    ptx::fence_proxy_async();
                    __syncwarp();
                }
                // (the barrier's one arrival is this arming, so copies that land before it cannot complete the phase)
                if (lane == 0) ptx::mbar_arrive_expect_tx(&full[st], (uint32_t)(n_tma * C::kSlotBytes));
                if (has_box && my_slot < n_tma) {
                    int page = my_page;
                    if (page < 0 || page >= p.num_pages) { dev_check(p, 400); page = 0; }
                    const int pg = u.layer * p.layer_pages + page;
                    if (vrole)
                        ptx::tma_load_5d(dst + my_slot * C::kSlotBytes, &tm_v, &full[st], 0, 0, 0, 0, pg * p.Hkv + u.g);
                    else
                        ptx::tma_load_5d(dst + my_slot * C::kSlotBytes, &tm_k, &full[st], 0, 0, 0, 0, pg * p.Hkv + u.g);
                }
                my_page = next_page;
            }
        }
        if (!ok && lane == 0) {
            // let copies already in flight land before the CTA's shared memory goes away
            const uint32_t ns = vrole ? VS : KR;
            const uint32_t back = it < ns ? it : ns;
            for (uint32_t j = it - back; j < it; ++j)
                ptx::mbar_wait(&full[j % ns], (j / ns) & 1, 200000000ll);
        }
    } else if (warp == 1) {
        // =========================================================================== Q K^T issuer
        if (lane == 0) {
            // descriptor words: the high words and the Q base are constants; per pair only low words move
            const uint32_t hi_q = ptx::umma_desc_hi_sw128(1024);
            const uint32_t hi_k = ptx::umma_desc_hi_sw128(C::kGroupStride);   // 8-token groups of a half: uniform over the pair's slots
            const uint32_t q_lo = ptx::umma_desc_lo(ptx::smem_u32(sQ), 16);
            const uint32_t k_lo = ptx::umma_desc_lo(ptx::smem_u32(sK), 16);
            // This one thread is busy for the whole tile period (its tcgen05.mma chain into one S buffer advances at
            // one instruction per ~100 cycles and holds it up meanwhile), so what it does between two chains is kept
            // short: ring stage, buffer and their parities are running counters, and the descriptor of a full tile is
            // made once.
            const uint32_t idesc_full = F8 ? umma_idesc_e4m3(kRows, kTileTok) : ptx::umma_idesc_bf16(kRows, kTileTok);
            uint32_t seg = 0;
            uint32_t st = 0, k_par = 0;            // K ring stage of the next tile and the parity its data completes
            uint32_t sb = 0, s_par = 1;            // S buffer of the next tile and the parity that says it is free
            bool ready = false;                    // both barriers of the next tile were seen complete already
            bool ok = true;
            long long x = x_begin;
            while (x < x_end && ok) {
                const Segment sg = make_segment(x, x_end, p, cumT, s_len, tiles_per_layer);
                if (!wait_bar(ctrl, &ctrl->q_full[seg & 1], (seg >> 1) & 1, p.wait_limit)) { timeout(p, ctrl, 20); ok = false; break; }
                const uint32_t q_seg = q_lo + (uint32_t)(((seg & 1) * q_buf_bytes) >> 4);
                ++seg;
                // one tile (a ring stage of four slots) per issue: each S buffer is scored as soon as the P V that read
                // it has completed, so the two softmax groups run half a period apart instead of in step
                int rem = sg.slots_all - sg.t_first * kStageSlots;               // slots left in the unit from this tile on
                // (parts hold whole pairs of tiles: two tiles per loop iteration halve what the loop itself costs this thread)
                auto issue_tile = [&](int rem_t) -> bool {
                    if (!ready && !wait_bar2(ctrl, &ctrl->k_full[st], k_par, &ctrl->s_free[sb], s_par, p.wait_limit)) return false;
                    ptx::tc_fence_after();
                    // the barriers of the tile after this one are polled now: the answers come back while this tile's
                    // chain holds the thread up (in the steady state both are complete long before)
                    const uint32_t st_n = (st + 1 == (uint32_t)KR) ? 0u : st + 1, k_par_n = k_par ^ (st_n == 0 ? 1u : 0u);
                    const uint32_t sb_n = (sb + 1) & (kSBufs - 1), s_par_n = s_par ^ (sb_n == 0 ? 1u : 0u);
                    const bool k_next = ptx::mbar_try_wait(&ctrl->k_full[st_n], k_par_n);
                    const bool s_next = ptx::mbar_try_wait(&ctrl->s_free[sb_n], s_par_n);
                    if (rem_t > 0) {                                                   // (a pair's second tile may be empty)
                        const uint32_t idesc = rem_t >= kStageSlots ? idesc_full
                                             : (F8 ? umma_idesc_e4m3(kRows, rem_t * kSlotTok) : ptx::umma_idesc_bf16(kRows, rem_t * kSlotTok));
                        const uint32_t kb = k_lo + st * (uint32_t)(C::kStageBytes >> 4);
                        const uint32_t d = tmem_base + sb * (uint32_t)kTileTok;
#pragma unroll
                        for (int kk = 0; kk < C::kRowBytes / 32; ++kk)          // 32 bytes of every row per instruction
                            umma_ss<F8>(d, q_seg + (uint32_t)(((kk >> 2) * p.q_half_bytes + (kk & 3) * 32) >> 4), hi_q,
                                               kb + (uint32_t)(((kk >> 2) * 1024 + (kk & 3) * 32) >> 4), hi_k, idesc, kk != 0);
                    }
                    ptx::umma_commit(&ctrl->s_full[sb]);
                    ptx::umma_commit(&ctrl->k_empty[st]);
                    st = st_n; k_par = k_par_n;
                    sb = sb_n; s_par = s_par_n;
                    ready = k_next && s_next;
                    return true;
                };
                for (int t = sg.t_first; t < sg.t_last; t += 2, rem -= 2 * kStageSlots) {
                    if (!issue_tile(rem) || !issue_tile(rem - kStageSlots)) { timeout(p, ctrl, 21); ok = false; break; }
                }
                x += sg.t_last - sg.t_first;
                if (!ok) break;
            }
        }
    } else if (warp == 2) {
        // =========================================================================== P V issuer
        if (lane == 0) {
            const uint32_t hi_v = ptx::umma_desc_hi_sw128(C::kGroupStride);                // the two 8-token groups of a slot
            const uint32_t v_lo = ptx::umma_desc_lo(ptx::smem_u32(sV), 1024);             // MN-major: LBO = next 64-column atom
            const uint32_t idesc_pv = (F8 ? umma_idesc_e4m3(kRows, D) : ptx::umma_idesc_bf16(kRows, D)) | (1u << 16);   // B operand MN-major
            uint32_t it = 0;
            int st = 0, sb = 0;                     // V ring stage and S / P buffer of the next tile, with their parities
            uint32_t v_par = 0, p_par = 0;
            bool ok = true;
            long long x = x_begin;
            uint32_t seg = 0;
            while (x < x_end && ok) {
                const Segment sg = make_segment(x, x_end, p, cumT, s_len, tiles_per_layer);
                // the accumulators of the previous part must have been read out by every softmax warp
                if (seg > 0 && (!wait_bar(ctrl, &ctrl->o_free, (seg - 1) & 1, p.wait_limit))) { timeout(p, ctrl, 24); ok = false; break; }
                ++seg;
                for (int t = sg.t_first; t < sg.t_last; ++t, ++x, ++it) {
                    const int pb = sb & 1;
                    if (!wait_bar2(ctrl, &ctrl->p_full[sb], p_par, &ctrl->v_full[st], v_par, p.wait_limit)) {
                        timeout(p, ctrl, 23); ok = false; break;
                    }
                    ptx::tc_fence_after();
                    const int n_sl = max(0, min(kStageSlots, sg.slots_all - t * kStageSlots));    // one 16-token step per slot
                    const uint32_t vb = v_lo + (uint32_t)((st * C::kStageBytes) >> 4);
                    const uint32_t pa = tmem_base + (uint32_t)(sb * kTileTok);       // P: 8 columns per 16-token step
                    // (e4m3: 32 tokens, two slots, per step; P is four codes per column, so a step is 8 columns either way)
                    constexpr int kStepSlots = F8 ? 2 : 1;
#pragma unroll
                    for (int k = 0; k < kStageSlots / kStepSlots; ++k)
                        if (k * kStepSlots < n_sl)
                            umma_ts<F8>(tmem_base + kTmemO + (uint32_t)(pb * D), pa + (uint32_t)(k * 8),
                                        vb + (uint32_t)(k * (kStepSlots * C::kSlotBytes / 16)), hi_v, idesc_pv, (t >= sg.t_first + 2) || (k != 0));
                    ptx::umma_commit(&ctrl->v_empty[st]);
                    ptx::umma_commit(&ctrl->s_free[sb]);
                    ptx::umma_commit(&ctrl->pv_done[pb]);
                    if (++st == VS) { st = 0; v_par ^= 1; }
                    sb = (sb + 1) & (kSBufs - 1);
                    if (sb == 0) p_par ^= 1;
                }
            }
        }
    } else {
        // =========================================================================== softmax / epilogue
        // Two groups of four warps (one thread per row each) take alternate tiles: group g owns the tiles whose
        // counter is g mod 2, with its own offset, running sum, P buffer and accumulator O_g in TMEM, exactly like
        // two split-KV partitions that are merged when the unit's part ends.  Nothing couples the groups per tile.
        const int w4 = warp & 3;                                   // TMEM lane quarter of this warp
        const int grp = (warp - 3) >> 2;                           // 0: warps 3..6, 1: warps 7..10
        uint32_t xph = 0;                                          // parity of the pair's exchange barrier
        const int row_in_blk = w4 * 32 + lane;
        const int rb_row0 = rb * p.rows_per_rb;
        const int rb_rows = min(p.rows_per_rb, p.rows - rb_row0);
        const bool row_ok = row_in_blk < rb_rows;
        const bool warp_has_rows = w4 * 32 < rb_rows;
        const int r_abs = rb_row0 + row_in_blk;                    // row within the unit: node * G + local head
        const int node = row_ok ? r_abs / p.G : 0, hl = row_ok ? r_abs % p.G : 0;
        const unsigned long long anc0 = tree.anc[node][0], anc1 = tree.anc[node][1];
        const uint32_t lane_base = tmem_base + ((uint32_t)(w4 * 32) << 16);
        const uint32_t o_mine = lane_base + kTmemO + (uint32_t)(grp * D);       // this group's accumulator
        constexpr int kDH = D / 2;                                 // output columns this warp finalises
        constexpr int kRowW = D + 4;                               // partial: D accumulator columns, then (max, sum) twice
        // both warps that share a TMEM quarter arrive (bounded wait, like every other wait in this kernel)
        auto pair_sync = [&]() -> bool {
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctrl->pair[w4]);
            const bool r = wait_bar(ctrl, &ctrl->pair[w4], xph, p.wait_limit);
            xph ^= 1;
            return r;
        };

        // this thread's half of its Q row goes into the swizzled A-operand tile `buf` by asynchronous 16-byte copies
        // (rows that do not exist are zero-filled); q_ready() later makes them visible to the tensor core
        auto stage_q = [&](const UnitPos& u, int buf) {
            const __nv_bfloat16* qrow = p.q + ((((size_t)u.layer * p.B + u.b) * p.n + node) * (size_t)p.Hq + u.g * p.G + hl) * D;
            uint8_t* q = sQ + buf * q_buf_bytes;
            const uint32_t src_bytes = row_ok ? 16u : 0u;
            if (row_in_blk * 128 >= p.q_half_bytes) return;        // the buffer holds no such row
            if constexpr (F8) {
                // this thread's 64 elements, divided by the Q scale and rounded to e4m3: four 16-byte chunks of the row
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 o = make_uint4(0, 0, 0, 0);
                    if (row_ok) {
                        const uint4 a = *reinterpret_cast<const uint4*>(qrow + grp * 64 + i * 16);
                        const uint4 b = *reinterpret_cast<const uint4*>(qrow + grp * 64 + i * 16 + 8);
                        auto cv = [&](uint32_t w0, uint32_t w1) -> uint32_t {      // two bf16 pairs -> four codes
                            // (a true fp32 division: the quotient decides the code)
                            return pack_e4m3x4(__fdiv_rn(__uint_as_float(w0 << 16), p.q_scale), __fdiv_rn(__uint_as_float(w0 & 0xffff0000u), p.q_scale),
                                               __fdiv_rn(__uint_as_float(w1 << 16), p.q_scale), __fdiv_rn(__uint_as_float(w1 & 0xffff0000u), p.q_scale));
                        };
                        o = make_uint4(cv(a.x, a.y), cv(a.z, a.w), cv(b.x, b.y), cv(b.z, b.w));
                    }
                    *reinterpret_cast<uint4*>(q + tile_off(row_in_blk, grp * 4 + i, p.q_half_bytes)) = o;
                }
                return;
            }
#pragma unroll
            for (int i = 0; i < D / 16; ++i) {
                const int chunk = grp * (D / 16) + i;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                             ::"r"(ptx::smem_u32(q + tile_off(row_in_blk, chunk, p.q_half_bytes))), "l"(qrow + chunk * 8), "r"(src_bytes) : "memory");
            }
        };
        auto q_ready = [&](int buf) {
            asm volatile("cp.async.wait_all;" ::: "memory");
            ptx::fence_proxy_async();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctrl->q_full[buf]);
        };

        uint32_t it = 0;
        bool ok = true;
        long long x = x_begin;
        Segment sg;
        // P of one tile from the row's 64 scores v[]: p = exp2(s*c - offset) as bf16 pairs, and the row sum in fp32
        float sc = p.scale_log2e;                                  // scores -> log2 units (e4m3: times the unit's Q and K scales)
        float vsc = 1.f;                                           // e4m3: the unit's V scale
        constexpr int kPW = F8 ? kTileTok / 4 : kTileTok / 2;      // 32-bit words of P per row and tile
        auto tile_p = [&](const float (&v)[kTileTok], float off_log2, uint32_t (&pk)[kPW]) -> float {
            const float o = (off_log2 == -INFINITY) ? 0.f : off_log2;       // nothing visible yet: every score is -inf
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
            if constexpr (F8) {
#pragma unroll
                for (int j = 0; j < kPW; ++j) {
                    const float e0 = ptx::ex2_approx(fmaf(v[4 * j], sc, -o)), e1 = ptx::ex2_approx(fmaf(v[4 * j + 1], sc, -o));
                    const float e2 = ptx::ex2_approx(fmaf(v[4 * j + 2], sc, -o)), e3 = ptx::ex2_approx(fmaf(v[4 * j + 3], sc, -o));
                    s0 += e0; s1 += e1; s2 += e2; s3 += e3;
                    pk[j] = pack_e4m3x4(e0, e1, e2, e3);
                }
                return (s0 + s1) + (s2 + s3);
            } else
#pragma unroll
            for (int j = 0; j < kTileTok / 2; j += 2) {
                pk[j] = exp2_pair(fmaf(v[2 * j], sc, -o), fmaf(v[2 * j + 1], sc, -o), s0, s1);
                pk[j + 1] = exp2_pair(fmaf(v[2 * j + 2], sc, -o), fmaf(v[2 * j + 3], sc, -o), s2, s3);
            }
            return (s0 + s1) + (s2 + s3);
        };
        auto tile_max = [&](const float (&v)[kTileTok]) -> float {
            float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
            for (int j = 0; j < kTileTok; j += 4) { m0 = max3(m0, v[j], v[j + 1]); m1 = max3(m1, v[j + 2], v[j + 3]); }
            return fmaxf(m0, m1);
        };

        uint32_t seg = 0;                                          // parts walked so far: Q buffer = seg & 1
        if (x < x_end) {
            sg = make_segment(x, x_end, p, cumT, s_len, tiles_per_layer);
            stage_q(sg.u, 0);
            q_ready(0);
        }
        while (x < x_end && ok) {
            const UnitPos u = sg.u;
            const bool whole_unit = (sg.t_first == 0 && sg.t_last == u.tiles_in_unit);
            float off_used = -INFINITY, l_run = 0.f;               // this group's offset (log2 units) and running sum
            if constexpr (F8) {
                sc = p.scale_log2e * p.q_scale * __ldg(p.k_scale + u.layer * p.Hkv + u.g);
                vsc = __ldg(p.v_scale + u.layer * p.Hkv + u.g);
            }
            // the part after this one: its Q goes into the other Q buffer now (every Q K^T that read that buffer
            // belongs to the part before this one and has completed), so the issuer can run on into the next unit
            Segment sg_next;
            const long long x_next = x + (sg.t_last - sg.t_first);
            const bool has_next = x_next < x_end;
            if (has_next) {
                sg_next = make_segment(x_next, x_end, p, cumT, s_len, tiles_per_layer);
                stage_q(sg_next.u, (seg + 1) & 1);
            }
            bool q_pending = has_next;

            // this group's tiles of the part: those whose counter has the group's parity
            const uint32_t it0 = it;
            for (int t = sg.t_first + (int)((it0 ^ (uint32_t)grp) & 1u); t < sg.t_last; t += 2) {
                it = it0 + (uint32_t)(t - sg.t_first);
                const int sb = it & (kSBufs - 1);
                if (!wait_bar(ctrl, &ctrl->s_full[sb], (it / kSBufs) & 1, p.wait_limit)) { timeout(p, ctrl, 30); ok = false; break; }
                ptx::tc_fence_after();
                float sum = 0.f;
                // visibility of this tile's columns for this row: all ones except in a unit's last pairs
                uint32_t cm0 = 0xffffffffu, cm1 = 0xffffffffu;
                if (t * kStageSlots + kStageSlots > sg.pages_full) {
                    cm0 = chunk_mask(t * kStageSlots, sg.pages_full, sg.pages_all, sg.slots_all, sg.len, anc0, anc1);
                    cm1 = chunk_mask(t * kStageSlots + 2, sg.pages_full, sg.pages_all, sg.slots_all, sg.len, anc0, anc1);
                }
                if (warp_has_rows) {
                    // one pass: the row's 64 scores are read once and P is computed against the offset in use, with no
                    // row maximum in the way; only the tile's SUM is watched
                    float v[kTileTok];
                    {
                        uint32_t r0[32], r1[32];
                        ptx::tmem_ld_32x32b_x32(lane_base + (uint32_t)(sb * kTileTok), r0);
                        ptx::tmem_ld_32x32b_x32(lane_base + (uint32_t)(sb * kTileTok + 32), r1);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; ++j) { v[j] = __uint_as_float(r0[j]); v[32 + j] = __uint_as_float(r1[j]); }
                    }
                    if ((cm0 & cm1) != 0xffffffffu) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (!((cm0 >> j) & 1u)) v[j] = -INFINITY;
                            if (!((cm1 >> j) & 1u)) v[32 + j] = -INFINITY;
                        }
                    }
                    // The offset (in log2 units) is set by the first tile in which the row sees anything: that tile's
                    // maximum.  (Before that every P was 0: nothing to rescale.)
                    if (__any_sync(0xffffffffu, off_used == -INFINITY)) {
                        const float mx = tile_max(v);
                        if (off_used == -INFINITY && mx > -INFINITY) off_used = mx * sc - PO::kBias;
                    }
                    uint32_t pk[kPW];
                    sum = tile_p(v, off_used, pk);
                    // The offset moves only when a tile's sum outgrows kSumLimit (an overflow makes the sum infinite, which
                    // counts): rare, and then this tile is redone against its own maximum after the accumulator and the
                    // running sum have been rescaled.  Whatever the offset, it is carried exactly through the sum and the
                    // final division.
                    const bool grow = !(sum <= PO::kSumLimit);
                    if (__any_sync(0xffffffffu, grow)) {
                        // this group's last P V (two tiles ago) must be complete before its accumulator is touched
                        if (it >= 2 && (!wait_bar(ctrl, &ctrl->pv_done[grp], ((it - 2) >> 1) & 1, p.wait_limit))) { timeout(p, ctrl, 33); ok = false; break; }
                        ptx::tc_fence_after();
                        const float off_next = grow ? tile_max(v) * sc - PO::kBias : off_used;
                        const float alpha = grow ? exp2f(off_used - off_next) : 1.f;
#pragma unroll 1
                        for (int c4 = 0; c4 < D / 32; ++c4) {
                            uint32_t r[32];
                            ptx::tmem_ld_32x32b_x32(o_mine + (uint32_t)(c4 * 32), r);
                            ptx::tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * alpha);
                            tmem_st_32x32b_x32(o_mine + (uint32_t)(c4 * 32), r);
                        }
                        l_run *= alpha;
                        off_used = off_next;
                        sum = tile_p(v, off_used, pk);
                    }
                    // P over the first 32 columns of the same S buffer (a thread only touches its own lane, and all of
                    // its scores are in registers)
                    if constexpr (F8) tmem_st_32x32b_x16(lane_base + (uint32_t)(sb * kTileTok), pk);
                    else tmem_st_32x32b_x32(lane_base + (uint32_t)(sb * kTileTok), pk);
                    tmem_st_wait();
                }
                l_run += sum;
                // Keep in step with this group's P V barrier: a parity wait can only tell apart two consecutive
                // phases, so a warp must never fall two completions behind it.  The P V of two tiles ago has
                // normally long completed here.
                if (it >= 2 && (!wait_bar(ctrl, &ctrl->pv_done[grp], ((it - 2) >> 1) & 1, p.wait_limit))) { timeout(p, ctrl, 34); ok = false; break; }
                // P is in tensor memory (and any O rescale too): the P V of this tile may go
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&ctrl->p_full[sb]);
                if (q_pending) { q_ready((seg + 1) & 1); q_pending = false; }
            }
            if (!ok) break;
            it = it0 + (uint32_t)(sg.t_last - sg.t_first);
            x = x_next;

            // (This part's Q buffer is overwritten at the start of the next part.  Every Q K^T that reads it has
            // completed by then: below, each group waits for the P V of its own last tile and then meets the other;
            // the P V of the part's last tile follows that tile's P, its S and so its Q K^T.  Waiting here on the
            // last tile's s_full instead would be wrong: the
            // issuer can run on into the next unit, and a second completion of that barrier would make a late
            // waiter's parity match the wrong phase.)
            if (q_pending) { q_ready((seg + 1) & 1); q_pending = false; }
            ++seg;

            // ---- end of this CTA's part of the unit: the two groups exchange (offset, sum), then each warp
            //      combines its half of the columns of both accumulators once the last P V is complete
            float* xc = xch + (size_t)row_in_blk * 4;              // [row][group][max, sum]
            xc[grp * 2] = off_used;
            xc[grp * 2 + 1] = l_run;
            // each group waits for the P V of its own last tile (the barrier it has kept in step with), then the
            // groups meet: past the meeting both accumulators are complete
            {
                const uint32_t j_last = (((it - 1) & 1) == (uint32_t)grp) ? it - 1 : it - 2;
                if (!wait_bar(ctrl, &ctrl->pv_done[grp], (j_last >> 1) & 1, p.wait_limit)) { timeout(p, ctrl, 32); ok = false; break; }
            }
            ptx::tc_fence_before();
            if (!pair_sync()) { timeout(p, ctrl, 35); ok = false; break; }
            ptx::tc_fence_after();
            const float m_a = xc[0], l_a = xc[1], m_b = xc[2], l_b = xc[3];
            const bool has_b = (sg.t_last - sg.t_first) >= 2;      // did the later-starting group see any tile?
            // group of the first tile of this part: the tile counter's parity when the part began
            const int g_first = (int)((it - (uint32_t)(sg.t_last - sg.t_first)) & 1);
            const bool has0 = has_b || g_first == 0, has1 = has_b || g_first == 1;
            const float M = fmaxf(has0 ? m_a : -INFINITY, has1 ? m_b : -INFINITY);
            const float w0 = (has0 && m_a != -INFINITY) ? exp2f(m_a - M) : 0.f;          // (offsets are in log2 units)
            const float w1 = (has1 && m_b != -INFINITY) ? exp2f(m_b - M) : 0.f;
            const float Lsum = w0 * (has0 ? l_a : 0.f) + w1 * (has1 ? l_b : 0.f);

            if (warp_has_rows) {
                __nv_bfloat16* orow = p.out + ((((size_t)u.layer * p.B + u.b) * p.n + node) * (size_t)p.Hq + u.g * p.G + hl) * D + grp * kDH;
                float* lse_ptr = (p.lse_out && grp == 0) ? p.lse_out + (((size_t)u.layer * p.B + u.b) * p.Hq + u.g * p.G + hl) * p.n + node : nullptr;
                const int slot = (sg.t_first > 0) ? 0 : 1;       // a unit that began before this CTA's range uses slot 0
                // partial layout [column][row]: a warp's store of one column is one contiguous 128-byte line;
                // each warp of a pair leaves its own copy of (max, sum) so that its columns stand alone
                float* my = p.partial + ((size_t)blockIdx.x * 2 + slot) * kRowW * kRows + row_in_blk;
                const float inv = vsc / Lsum;                      // (e4m3: V codes times the unit's V scale)
                // combined accumulator columns [grp*kDH, (grp+1)*kDH) of both groups' O, 32 at a time
#pragma unroll 1
                for (int c4 = 0; c4 < kDH / 32; ++c4) {
                    float acc[32];
                    {
                        uint32_t ra[32];
                        if (has0) {
                            ptx::tmem_ld_32x32b_x32(lane_base + kTmemO + (uint32_t)(grp * kDH + c4 * 32), ra);
                            ptx::tmem_ld_wait();
                        }
#pragma unroll
                        for (int j = 0; j < 32; ++j) acc[j] = (has0 && m_a != -INFINITY) ? w0 * __uint_as_float(ra[j]) : 0.f;   // (an accumulator no P V wrote may hold anything)
                        if (has1) {
                            ptx::tmem_ld_32x32b_x32(lane_base + kTmemO + (uint32_t)(D + grp * kDH + c4 * 32), ra);
                            ptx::tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 32; ++j) acc[j] = (m_b != -INFINITY) ? fmaf(w1, __uint_as_float(ra[j]), acc[j]) : acc[j];
                        }
                    }
                    if (whole_unit) {
                        if (row_ok) {
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                uint4 v;
                                v.x = pack_bf16(acc[j * 8 + 0] * inv, acc[j * 8 + 1] * inv);
                                v.y = pack_bf16(acc[j * 8 + 2] * inv, acc[j * 8 + 3] * inv);
                                v.z = pack_bf16(acc[j * 8 + 4] * inv, acc[j * 8 + 5] * inv);
                                v.w = pack_bf16(acc[j * 8 + 6] * inv, acc[j * 8 + 7] * inv);
                                *reinterpret_cast<uint4*>(orow + c4 * 32 + j * 8) = v;
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) my[(size_t)(grp * kDH + c4 * 32 + j) * kRows] = acc[j] * vsc;
                    }
                }
                // both accumulators have been read by this warp: the next unit's P V may overwrite them once all have
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&ctrl->o_free);
                if (whole_unit) {
                    if (lse_ptr && row_ok) *lse_ptr = M * kLn2 + logf(Lsum);
                } else {
                    // ---- the unit is cut across CTA groups: this part's (max, sum, accumulator) is left for the merge
                    //      kernel that follows; nothing here waits for another CTA
                    my[(size_t)(D + 2 * grp) * kRows] = M;
                    my[(size_t)(D + 2 * grp + 1) * kRows] = Lsum;
                }
            } else {
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&ctrl->o_free);
            }
            // the exchange words are rewritten at the end of the next part: the partner must have read them
            if (!pair_sync()) { timeout(p, ctrl, 36); ok = false; break; }
            if (has_next) sg = sg_next;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");      // (only an aborted run can still have copies in flight here)
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// Merge of the units that the partition cut across CTA groups.  One block per (inner boundary, row block).  A unit
// cut by k boundaries left k + 1 (max, sum, accumulator) records, like split-KV partials; the k blocks of those
// boundaries share its merge by output columns (8-column chunks dealt round-robin), each combining all parts of its
// columns in group order, so a unit that many CTAs shared (few units per launch, long contexts) is not merged by one
// block alone.  Blocks whose boundary coincides with a unit boundary have nothing to do.
constexpr int kMergeThreads = 512;        // 128 rows x 4 column quarters
constexpr int kMergeMaxGroups = 512;      // groups whose first tiles fit the lookup table (more: computed on demand)
template <int D>
__global__ void __launch_bounds__(kMergeThreads) attn_merge_kernel(const AttnParams p) {
    __shared__ int cumT[kMaxBatch + 1];
    __shared__ int s_len[kMaxBatch];
    const int tid = threadIdx.x;
    for (int b = tid; b < p.B; b += kMergeThreads) {
        const int len = p.prefix_len[b];
        s_len[b] = len < 0 ? 0 : (len > p.max_pages * kSlotTok ? p.max_pages * kSlotTok : len);
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        cumT[0] = 0;
        for (int b = 0; b < p.B; ++b) {
            const int slots = (s_len[b] + kSlotTok - 1) / kSlotTok + p.tree_slots;
            acc += 2 * ((slots + 2 * kStageSlots - 1) / (2 * kStageSlots));
            cumT[b + 1] = acc;
        }
    }
    __syncthreads();
    const Partition part = make_partition(p, cumT);
    const int g = blockIdx.x + 1, rb = blockIdx.y;
    // A block with nothing to merge must still wait for the attention kernel: the kernel behind this one in the stream
    // only waits for THIS grid to complete, so a grid whose blocks all left early would let it read attention outputs
    // that are still being written.
    if (g >= part.n_groups || part.total_tiles >= (1ll << 31)) { ptx::grid_dep_wait(); return; }
    const long long x = group_begin(part, g, p, cumT);
    const UnitPos u = locate(x, p, cumT, part.tiles_per_layer);
    if (u.tile_in_unit == 0) { ptx::grid_dep_wait(); return; }                  // the boundary is a unit boundary (block-uniform)
    // every group's first tile, computed side by side (a unit shared by many groups is looked up from here instead of
    // by a chain of dependent calls)
    __shared__ long long s_begin[kMergeMaxGroups];
    const bool tabled = part.n_groups <= kMergeMaxGroups;
    if (tabled) {
        for (int t = tid; t < part.n_groups; t += kMergeThreads) s_begin[t] = group_begin(part, t, p, cumT);
        __syncthreads();
    }
    auto begin_of = [&](int t) -> long long { return tabled ? s_begin[t] : group_begin(part, t, p, cumT); };
    // the groups ga..gb hold this unit's parts; the blocks of the boundaries ga+1..gb share the merge by columns
    int ga = g - 1;
    while (ga > 0 && begin_of(ga) > u.unit_first_tile) --ga;
    int gb = g;
    const long long unit_last = u.unit_first_tile + u.tiles_in_unit - 1;
    while (gb + 1 < part.n_groups && begin_of(gb + 1) <= unit_last) ++gb;
    const int parts = gb - ga + 1;
    const int n_blocks = parts - 1, j_blk = g - (ga + 1);
    // launched with programmatic stream serialization: everything above overlaps the attention kernel's tail;
    // its records (and the outputs this block overwrites) are only touched after it has completed
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();

    constexpr int kRowW = D + 4;
    constexpr int kChunks = D / 8;                                              // 8 output columns = one 16-byte store
    constexpr int kPer = (kChunks + 3) / 4;                                     // chunks per thread when one block has them all
    const int row = tid & (kRows - 1), cq = tid >> 7;
    const int rb_row0 = rb * p.rows_per_rb;
    const int rb_rows = min(p.rows_per_rb, p.rows - rb_row0);
    if (row >= rb_rows) return;
    const int r_abs = rb_row0 + row, node = r_abs / p.G, hl = r_abs % p.G;
    // chunk c belongs to block c mod n_blocks; inside the block its chunks go round the four thread quarters
    int chunk[kPer];
    bool any = false;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        chunk[i] = j_blk + (cq + 4 * i) * n_blocks;
        any |= chunk[i] < kChunks;
    }
    const bool writes_lse = p.lse_out && j_blk == 0 && cq == 0;
    if (!any && !writes_lse) return;
    // group ga holds the unit's first tile (its record is in slot 1), the later groups began inside the unit (slot 0)
    auto part_of = [&](int k) -> const float* {
        return p.partial + ((size_t)((ga + k) * p.n_rb + rb) * 2 + (k == 0 ? 1 : 0)) * kRowW * kRows + row;
    };
    float Mm = -INFINITY;
#pragma unroll 4
    for (int k = 0; k < parts; ++k) Mm = fmaxf(Mm, __ldcg(part_of(k) + (size_t)D * kRows));
    float Lm = 0.f;
    float acc[kPer][8];
#pragma unroll
    for (int i = 0; i < kPer; ++i)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[i][c] = 0.f;
    if (n_blocks >= 4) {
        // many parts, at most one chunk per thread: six parts' loads in flight at a time (same order of additions)
        if (chunk[0] < kChunks || writes_lse) {
            const bool has = chunk[0] < kChunks;
            const int c0 = has ? chunk[0] * 8 : 0;
#pragma unroll 6
            for (int k = 0; k < parts; ++k) {
                const float* src = part_of(k);
                const float pm = __ldcg(src + (size_t)D * kRows);
                const float wgt = (pm == -INFINITY) ? 0.f : exp2f(pm - Mm);
                Lm = fmaf(wgt, __ldcg(src + (size_t)(D + 1) * kRows), Lm);
                if (has) {
#pragma unroll
                    for (int c = 0; c < 8; ++c) acc[0][c] = fmaf(wgt, __ldcg(src + (size_t)(c0 + c) * kRows), acc[0][c]);
                }
            }
        }
    } else
#pragma unroll 2
    for (int k = 0; k < parts; ++k) {
        const float* src = part_of(k);
        const float pm = __ldcg(src + (size_t)D * kRows);
        const float wgt = (pm == -INFINITY) ? 0.f : exp2f(pm - Mm);
        Lm = fmaf(wgt, __ldcg(src + (size_t)(D + 1) * kRows), Lm);
#pragma unroll
        for (int i = 0; i < kPer; ++i)
            if (chunk[i] < kChunks) {
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[i][c] = fmaf(wgt, __ldcg(src + (size_t)(chunk[i] * 8 + c) * kRows), acc[i][c]);
            }
    }
    const float inv = 1.f / Lm;
    __nv_bfloat16* orow = p.out + ((((size_t)u.layer * p.B + u.b) * p.n + node) * (size_t)p.Hq + u.g * p.G + hl) * D;
#pragma unroll
    for (int i = 0; i < kPer; ++i)
        if (chunk[i] < kChunks) {
            uint4 v;
            v.x = pack_bf16(acc[i][0] * inv, acc[i][1] * inv);
            v.y = pack_bf16(acc[i][2] * inv, acc[i][3] * inv);
            v.z = pack_bf16(acc[i][4] * inv, acc[i][5] * inv);
            v.w = pack_bf16(acc[i][6] * inv, acc[i][7] * inv);
            *reinterpret_cast<uint4*>(orow + chunk[i] * 8) = v;
        }
    if (writes_lse)
        p.lse_out[(((size_t)u.layer * p.B + u.b) * p.Hq + u.g * p.G + hl) * p.n + node] = Mm * kLn2 + logf(Lm);
}

}  // namespace

mirror_status mirror_attn_launch(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const MirrorTreeInfo& ti,
                                 const void* q, const void* k_new, const void* v_new, void* out, float* lse_out,
                                 float* partial_ws, cudaStream_t stream, const MirrorAttnFp8* f8) {
    const int D = ctx->desc.head_dim, Hkv = ctx->desc.n_kv_heads, Hq = ctx->desc.n_q_heads;
    AttnParams p;
    p.L = kv->num_layers; p.B = tree->batch; p.n = ti.n; p.Hq = Hq; p.Hkv = Hkv; p.G = Hq / Hkv;
    p.rows = p.G * p.n;
    p.n_rb = (p.rows + kRows - 1) / kRows;
    p.rows_per_rb = (p.rows + p.n_rb - 1) / p.n_rb;
    p.n_groups = ctx->num_sms / p.n_rb;
    if (ctx->tune.attn_groups >= 1 && ctx->tune.attn_groups <= p.n_groups) p.n_groups = ctx->tune.attn_groups;
    if (p.n_groups < 1) return MIRROR_ERR_SHAPE;
    p.snap_cap = ctx->tune.attn_snap;
    p.whole_units = ctx->tune.attn_whole_units;
    p.wait_limit = ctx->tune.wait_limit_cycles;
    p.stall_after = (ctx->tune.test_stall_after >= 0 && ctx->tune.test_stall_attn_left-- > 0) ? ctx->tune.test_stall_after : -1;
    p.max_pages = kv->max_pages_per_req; p.num_pages = kv->num_pages;
    const int64_t page_elems = (int64_t)Hkv * kSlotTok * D;
    if (kv->layer_stride % page_elems != 0) return MIRROR_ERR_UNSUPPORTED;
    if (f8 && (D != 128 || !f8->k_scale || !f8->v_scale || !(f8->q_scale > 0.f))) return f8 && D != 128 ? MIRROR_ERR_UNSUPPORTED : MIRROR_ERR_ARG;
    p.k_scale = f8 ? f8->k_scale : nullptr;
    p.v_scale = f8 ? f8->v_scale : nullptr;
    p.q_scale = f8 ? f8->q_scale : 1.f;
    p.layer_pages = (int)(kv->layer_stride / page_elems);
    p.tree_slots = (p.n + kSlotTok - 1) / kSlotTok;
    p.q_half_bytes = ((p.rows_per_rb + 7) / 8) * 8 * 128;
    p.scale = ctx->scale;
    p.scale_log2e = ctx->scale * 1.4426950408889634f;
    p.page_table = kv->page_table; p.prefix_len = kv->prefix_len;
    p.q = (const __nv_bfloat16*)q;
    p.k_pool = (const __nv_bfloat16*)kv->k_pool; p.v_pool = (const __nv_bfloat16*)kv->v_pool;
    p.k_new = (const __nv_bfloat16*)k_new; p.v_new = (const __nv_bfloat16*)v_new;
    p.out = (__nv_bfloat16*)out; p.lse_out = lse_out;
    p.partial = partial_ws; p.status = ctx->d_status;
    if (p.B > kMaxBatch) return MIRROR_ERR_SHAPE;

    AttnTree at;
    memcpy(at.anc, ti.anc, sizeof at.anc);

    CUtensorMap tm_k, tm_v;
    {
        // pool viewed as (64 columns, 8 tokens, D/64 halves, 2 token groups, (layer*page)*head): one box is one page of
        // one head, landing as [token / 8][half][token % 8][128 B] (see kv_slot_off)
        // (an e4m3 pool is described through the same 16-bit map: 64 "columns" are the 128 bytes of a row's only half)
        const uint64_t total_pages = (uint64_t)(p.L - 1) * p.layer_pages + p.num_pages;
        const uint64_t row_bytes = (uint64_t)D * (f8 ? 1 : 2);
        const uint64_t dims[5] = {64, 8, row_bytes / 128, 2, total_pages * (uint64_t)Hkv};
        const uint64_t strides[4] = {row_bytes, 128, 8 * row_bytes, kSlotTok * row_bytes};
        const uint32_t box[5] = {64, 8, (uint32_t)(row_bytes / 128), 2, 1};
        mirror_status st = mirror_make_tmap(ctx, &tm_k, kv->k_pool, 5, dims, strides, box);
        if (st != MIRROR_OK) return st;
        st = mirror_make_tmap(ctx, &tm_v, kv->v_pool, 5, dims, strides, box);
        if (st != MIRROR_OK) return st;
    }
    const int grid = p.n_groups * p.n_rb;
    // ring depths: the deepest pair (K, V) that fits beside the Q buffers
    constexpr size_t kSmemLimit = 232448;       // 227 KB
    auto launch = [&](auto d_tag, auto f8_tag) -> mirror_status {
        constexpr int DD = decltype(d_tag)::value;
        constexpr bool FF = decltype(f8_tag)::value;
        using C = Cfg<DD, FF>;
        int ks = 4, vs = 4;
        if (C::smem_bytes(p.q_half_bytes, 6, 4) <= kSmemLimit) ks = 6;
        if (C::smem_bytes(p.q_half_bytes, 6, 6) <= kSmemLimit) vs = 6;
        if (ctx->tune.attn_ring) { ks = ctx->tune.attn_ring / 10; vs = ctx->tune.attn_ring % 10; }
        if (!((ks == 4 || ks == 6) && (vs == 4 || (vs == 6 && ks == 6)))) return MIRROR_ERR_ARG;
        const size_t smem = C::smem_bytes(p.q_half_bytes, ks, vs);
        if (smem > kSmemLimit) return MIRROR_ERR_UNSUPPORTED;
        auto go = [&](auto kern) -> mirror_status {
            MIRROR_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit));
            MIRROR_CUDA_OK(mirror_launch_pdl(kern, dim3(grid), dim3(kThreads), smem, stream, tm_k, tm_v, at, p));
            return MIRROR_OK;
        };
        if (ks == 6 && vs == 6) return go(attn_verify_kernel<DD, 6, 6, FF>);
        if constexpr (!FF) {
            if (ks == 6) return go(attn_verify_kernel<DD, 6, 4, false>);
            return go(attn_verify_kernel<DD, 4, 4, false>);
        }
        return MIRROR_ERR_ARG;
    };
    mirror_status lst = f8 ? launch(std::integral_constant<int, 128>{}, std::true_type{})
                      : (D == 128) ? launch(std::integral_constant<int, 128>{}, std::false_type{})
                                   : launch(std::integral_constant<int, 64>{}, std::false_type{});
    if (lst != MIRROR_OK) return lst;
    ctx->launches += 1;
    MIRROR_CUDA_OK(cudaGetLastError());
    // One request: all units have the same length whatever it is, so the host can tell when the partition gives every
    // group whole units (each unit holds at least one pair of tiles, so there are at least L * Hkv pairs): nothing is cut
    // and the merge kernel has nothing to do.
    const bool no_cuts = p.whole_units && p.B == 1 && (long long)p.L * p.Hkv >= p.n_groups &&
                         whole_unit_groups(p.n_groups, (long long)p.L * p.B * p.Hkv) > 0;
    if (p.n_groups > 1 && !no_cuts) {
        // which units the partition cut is only known on the device (it depends on the prefix lengths)
        const dim3 mgrid((unsigned)(p.n_groups - 1), (unsigned)p.n_rb);
        if (D == 128) MIRROR_CUDA_OK(mirror_launch_pdl(attn_merge_kernel<128>, mgrid, dim3(kMergeThreads), 0, stream, p));
        else MIRROR_CUDA_OK(mirror_launch_pdl(attn_merge_kernel<64>, mgrid, dim3(kMergeThreads), 0, stream, p));
        ctx->launches += 1;
        MIRROR_CUDA_OK(cudaGetLastError());
    }
    return MIRROR_OK;
}
