// Acceptance, branch selection, emitted tokens and reuse lookup (Sec. 3.1; Eq. 3 / Eq. 10).
//
// One thread block per request.  Warps take branches round-robin; lane j of a warp tests the node at
// depth j+1 of its branch, a ballot gives the number of leading passes (the acceptance operator of
// Eq. 3 applied to that branch).  Thread 0 then picks the longest branch (lowest index on ties) and the
// deciding row R.  Greedy mode emits argmax[R]; speculative-sampling mode draws the extra token by an
// inverse-CDF search over the vocabulary that the whole block cooperates on, all in fp64.
#include <cooperative_groups.h>

#include "mirror_internal.h"

namespace {

constexpr int kThreads = 1024;

struct AcceptTreeParams {
    int n, n_branches, gamma;
    unsigned char parent[MIRROR_MAX_NODES];
    unsigned char path[MIRROR_MAX_BRANCHES][MIRROR_MAX_DEPTH];
    unsigned char path_len[MIRROR_MAX_BRANCHES];
};

struct AcceptArgs {
    int mode, emit_bonus, V, n_cand;
    double inv_T;
    const int32_t* tokens;
    const int32_t* target_argmax;
    const float* logits;
    const float* lse;
    const float* q_probs;
    const float* u_accept;
    const float* u_resample;
    const int32_t* cand_ids;
    mirror_accept_out out;
    double* tree_scratch;          // nullable fp64 [B, 2, V]: running distribution of the tree rule
    int* status;
};

__device__ __forceinline__ double warp_excl_scan(double v, int lane, double* total) {
    double inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    *total = __shfl_sync(0xffffffffu, inc, 31);
    return inc - v;
}

__global__ void __launch_bounds__(kThreads, 1)
accept_select_kernel(const __grid_constant__ AcceptTreeParams tp, const AcceptArgs a) {
    __shared__ int s_len[MIRROR_MAX_BRANCHES];
    __shared__ int s_A, s_best, s_R, s_rej_node, s_extra, s_last_pos, s_seg;
    __shared__ double s_seg_p[kThreads], s_seg_r[kThreads];
    __shared__ double s_thr, s_excl;
    __shared__ int s_use_res;

    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = tp.n, V = a.V;
    const int32_t* tok = a.tokens + (size_t)b * n;
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();

    for (int br = warp; br < tp.n_branches; br += kThreads / 32) {
        const int len = tp.path_len[br];
        bool pass = true;
        if (lane < len) {
            const int c = tp.path[br][lane];
            const int r = tp.parent[c];
            const int x = tok[c];
            if (a.mode == MIRROR_ACCEPT_GREEDY) {
                pass = (x == a.target_argmax[(size_t)b * n + r]);
            } else if (x < 0 || x >= V) {
                pass = false;
                if (atomicCAS(a.status, 0, MIRROR_DEV_CHECK) == 0) atomicExch(a.status + 1, 100 + c);   // first error wins
            } else {
                const size_t row = (size_t)b * n + r;
                const double p = exp((double)a.logits[row * V + x] * a.inv_T - (double)a.lse[row]);
                const double lhs = (double)a.u_accept[(size_t)b * n + c] *
                                   (double)a.q_probs[((size_t)b * (n - 1) + (c - 1)) * V + x];
                pass = (lhs <= p);
            }
        }
        const unsigned fail = __ballot_sync(0xffffffffu, lane < len && !pass);
        if (lane == 0) s_len[br] = fail ? (__ffs(fail) - 1) : len;
    }
    __syncthreads();

    if (tid == 0) {
        int A = 0, best = 0;
        for (int i = 0; i < tp.n_branches; ++i)
            if (s_len[i] > A) { A = s_len[i]; best = i; }
        const int R = (A == 0) ? 0 : tp.path[best][A - 1];
        const bool rejected = tp.n_branches > 0 && A < tp.path_len[best];
        s_A = A; s_best = best; s_R = R;
        s_rej_node = rejected ? tp.path[best][A] : -1;
        s_extra = -1; s_last_pos = -1; s_seg = -1;
    }
    __syncthreads();
    const int A = s_A, best = s_best, R = s_R, rej_node = s_rej_node;
    const bool have_extra = (rej_node >= 0) || tp.n_branches == 0 || a.emit_bonus != 0;

    if (have_extra) {
        if (a.mode == MIRROR_ACCEPT_GREEDY) {
            if (tid == 0) s_extra = a.target_argmax[(size_t)b * n + R];
        } else {
            // inverse-CDF draw over the vocabulary from max(0, p - q') (rejection) or p (bonus), fp64
            const size_t rowR = (size_t)b * n + R;
            const float* lr = a.logits + rowR * V;
            const double lseR = (double)a.lse[rowR];
            const float* qc = (rej_node >= 0) ? a.q_probs + ((size_t)b * (n - 1) + (rej_node - 1)) * V : nullptr;
            const int S = (V + kThreads - 1) / kThreads;
            const int v0 = min(tid * S, V), v1 = min(v0 + S, V);
            double sp = 0.0, sr = 0.0;
            for (int v = v0; v < v1; ++v) {
                const double p = exp((double)lr[v] * a.inv_T - lseR);
                sp += p;
                if (qc) {
                    const double res = p - (double)qc[v];
                    sr += (res > 0.0) ? res : 0.0;
                }
            }
            s_seg_p[tid] = sp;
            s_seg_r[tid] = sr;
            __syncthreads();
            if (warp == 0) {
                // totals in segment order, then the first segment whose inclusive prefix passes the threshold
                double lp = 0.0, lres = 0.0;
                for (int k = 0; k < 32; ++k) { lp += s_seg_p[lane * 32 + k]; lres += s_seg_r[lane * 32 + k]; }
                double tot_p, tot_r;
                const double ex_p = warp_excl_scan(lp, lane, &tot_p);
                const double ex_r = warp_excl_scan(lres, lane, &tot_r);
                const int use_res = (qc != nullptr) && (tot_r > 0.0);
                const double thr = (double)a.u_resample[(size_t)b * n + R] * (use_res ? tot_r : tot_p);
                double run = use_res ? ex_r : ex_p;
                int found = -1;
                double found_excl = 0.0;
                for (int k = 0; k < 32; ++k) {
                    const double seg = use_res ? s_seg_r[lane * 32 + k] : s_seg_p[lane * 32 + k];
                    if (found < 0 && run + seg > thr) { found = lane * 32 + k; found_excl = run; }
                    run += seg;
                }
                const unsigned m = __ballot_sync(0xffffffffu, found >= 0);
                if (m) {
                    const int src = __ffs(m) - 1;
                    if (lane == src) { s_seg = found; s_excl = found_excl; }
                }
                if (lane == 0) { s_thr = thr; s_use_res = use_res; }
            }
            __syncthreads();
            const int use_res = s_use_res;
            if (s_seg >= 0) {
                if (tid == s_seg) {
                    const double thr = s_thr, excl = s_excl;
                    double loc = 0.0;
                    int pick = v1 - 1;
                    for (int v = v0; v < v1; ++v) {
                        const double p = exp((double)lr[v] * a.inv_T - lseR);
                        double mass = p;
                        if (use_res) { const double res = p - (double)qc[v]; mass = (res > 0.0) ? res : 0.0; }
                        loc += mass;
                        if (excl + loc > thr) { pick = v; break; }
                    }
                    s_extra = pick;
                }
            } else {
                // rounding left no crossing: take the last id with positive mass
                int last = -1;
                for (int v = v0; v < v1; ++v) {
                    const double p = exp((double)lr[v] * a.inv_T - lseR);
                    double mass = p;
                    if (use_res) { const double res = p - (double)qc[v]; mass = (res > 0.0) ? res : 0.0; }
                    if (mass > 0.0) last = v;
                }
                if (last >= 0) atomicMax(&s_last_pos, last);
                __syncthreads();
                if (tid == 0) s_extra = s_last_pos;
            }
        }
    }
    __syncthreads();

    const int gamma = tp.gamma;
    if (tid <= gamma) {
        int e = -1;
        if (tid < A) e = tok[tp.path[best][tid]];
        else if (tid == A && have_extra) e = s_extra;
        a.out.emitted[(size_t)b * (gamma + 1) + tid] = e;
        if (tid < gamma) a.out.accepted_nodes[(size_t)b * gamma + tid] = (tid < A) ? (int)tp.path[best][tid] : -1;
    }
    if (tid == 0) {
        a.out.n_accepted[b] = A;
        a.out.best_branch[b] = best;
        a.out.decide_row[b] = R;
        a.out.n_emitted[b] = A + (have_extra ? 1 : 0);
        int slot = -1;
        if (have_extra && a.cand_ids)
            for (int k = 0; k < a.n_cand; ++k)
                if (a.cand_ids[((size_t)b * n + R) * a.n_cand + k] == s_extra) { slot = k; break; }
        a.out.reuse_slot[b] = slot;
    }
}

// ---------------------------------------------------------------------------------------------------
// Lossless acceptance over a token tree: sequential multi-round rejection over the siblings of each accepted
// row (the speculative-sampling rule of Sec. 3.1 applied to sibling sets, for tree drafts).  A cluster of
// kTreeCluster CTAs per request walks down from the root, every CTA holding one contiguous slice of the vocabulary.
// At row r the current distribution m starts as the target's p_r; the children of r are tested in node order
// against m: child c (token x, draft distribution q_c) passes iff u_accept[c] * q_c[x] <= m[x] and the walk moves to
// c; a child that fails turns m into the normalised residual max(0, m - q_c).  m[v] is either re-evaluated from the
// logits, the rejected siblings' q rows and their normalisers Z_i, or -- when the caller's workspace has room --
// kept in fp64 scratch memory (two buffers, so that a residual without mass can be dropped); both follow the
// definition's operation order per element.  A rejection costs one pass over the vocabulary for Z, the final draw
// one more; the CTAs exchange their slice sums through distributed shared memory and add them in rank order, so
// all of them see identical numbers, take identical decisions and stay in step (one hardware cluster barrier per
// pass, nothing spins).
// ---------------------------------------------------------------------------------------------------
constexpr int kMaxRejected = MIRROR_MAX_BRANCHES;     // siblings rejected at one row
constexpr int kTreeCluster = 8;                       // CTAs per request

__global__ void __launch_bounds__(kThreads, 1)
accept_tree_kernel(const __grid_constant__ AcceptTreeParams tp, const AcceptArgs a) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ double s_seg[kThreads];
    __shared__ double s_Z[kMaxRejected];
    __shared__ int s_rej[kMaxRejected];
    __shared__ int s_path[MIRROR_MAX_DEPTH];
    __shared__ double s_slice[2];                     // this CTA's slice sum of the current pass (by pass parity): read by peers
    __shared__ double s_excl;
    __shared__ int s_pass, s_found, s_extra, s_last;

    const int rank = (int)cluster.block_rank();
    const int b = blockIdx.x / kTreeCluster, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = tp.n, V = a.V;
    const int32_t* tok = a.tokens + (size_t)b * n;
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    // this CTA's slice of the vocabulary and this thread's contiguous segment of it
    const int Vs = (V + kTreeCluster - 1) / kTreeCluster;
    const int s0 = min(rank * Vs, V), s1 = min(s0 + Vs, V);
    const int S = (Vs + kThreads - 1) / kThreads;
    const int v0 = min(s0 + tid * S, s1), v1 = min(v0 + S, s1);

    int r = 0, A = 0, n_rej = 0, n_children = 0;
    uint32_t pass_no = 0;                          // vocabulary passes so far (identical in every CTA)
    double* const buf0 = a.tree_scratch ? a.tree_scratch + (size_t)b * 2 * V : nullptr;
    double* const buf1 = buf0 ? buf0 + V : nullptr;
    int cur = 0;                                   // buffer that holds the current residual (when n_rej > 0)
    double inv_Z = 1.0;                            // 1 / Z of the last effective rejection
    // m[v] at row r after the rejections recorded so far
    auto mass = [&](const float* lr, double lse_r, int v) -> double {
        if (buf0 && n_rej > 0) return (cur ? buf1 : buf0)[v] * inv_Z;       // (times 1/Z: one rounding away from the quotient)
        double m = exp((double)lr[v] * a.inv_T - lse_r);
        for (int i = 0; i < n_rej; ++i) {
            const double res = m - (double)a.q_probs[((size_t)b * (n - 1) + (s_rej[i] - 1)) * V + v];
            m = ((res > 0.0) ? res : 0.0) / s_Z[i];
        }
        return m;
    };
    // Sum of f over the whole vocabulary in a fixed order: per-thread partial sums over this CTA's slice (contiguous
    // segments, whose sums the inverse-CDF search reuses, or ids interleaved over the threads, which keeps a warp's
    // loads in one line), warp 0 adds them in order, then every CTA adds the eight slice sums in rank order.
    // excl_out: sum of the slices before this CTA's.
    auto cluster_total = [&](auto f, bool contiguous, double* excl_out) -> double {
        double part = 0.0;
        if (contiguous) {
            for (int v = v0; v < v1; ++v) part += f(v);
        } else {
            double p0 = 0.0, p1 = 0.0, p2 = 0.0, p3 = 0.0;
            int v = s0 + tid;
            for (; v + 3 * kThreads < s1; v += 4 * kThreads) {
                p0 += f(v); p1 += f(v + kThreads); p2 += f(v + 2 * kThreads); p3 += f(v + 3 * kThreads);
            }
            for (; v < s1; v += kThreads) p0 += f(v);
            part = (p0 + p1) + (p2 + p3);
        }
        s_seg[tid] = part;
        __syncthreads();
        const int par = pass_no & 1;
        if (warp == 0) {
            double lp = 0.0;
            for (int k = 0; k < 32; ++k) lp += s_seg[lane * 32 + k];
            double tot;
            warp_excl_scan(lp, lane, &tot);
            if (lane == 0) s_slice[par] = tot;
        }
        // (release / acquire at cluster scope: the slice sums and, with scratch memory, the residuals the peers wrote
        // to global memory in this pass are visible after the barrier.  A buffer of this parity is written again two
        // passes later, after every peer has passed the barrier in between and so finished reading it.)
        cluster.sync();
        double tot = 0.0, excl = 0.0;
        for (int c = 0; c < kTreeCluster; ++c) {
            if (c == rank) excl = tot;
            tot += *cluster.map_shared_rank(&s_slice[par], c);
        }
        ++pass_no;
        if (excl_out) *excl_out = excl;
        return tot;
    };

    for (;;) {
        const size_t row = (size_t)b * n + r;
        const float* lr = a.logits + row * V;
        const double lse_r = (double)a.lse[row];
        n_rej = 0;
        n_children = 0;
        int next = -1;
        for (int c = r + 1; c < n; ++c) {
            if (tp.parent[c] != r) continue;
            ++n_children;
            const float* qc = a.q_probs + ((size_t)b * (n - 1) + (c - 1)) * V;
            if (tid == 0) {
                // (every CTA evaluates the test itself, from numbers that are identical in all of them)
                const int x = tok[c];
                int pass = 0;
                if (x < 0 || x >= V) {
                    if (atomicCAS(a.status, 0, MIRROR_DEV_CHECK) == 0) atomicExch(a.status + 1, 100 + c);   // first error wins
                } else {
                    const double lhs = (double)a.u_accept[(size_t)b * n + c] * (double)qc[x];
                    pass = (lhs <= mass(lr, lse_r, x)) ? 1 : 0;
                }
                s_pass = pass;
            }
            __syncthreads();
            if (s_pass) { next = c; break; }
            // rejected: normaliser of the residual (a residual without mass leaves m as it is)
            double* const nxt = !buf0 ? nullptr : ((n_rej > 0 && cur == 0) ? buf1 : buf0);      // the buffer not in use
            const double Z = cluster_total([&](int v) {
                double res = mass(lr, lse_r, v) - (double)qc[v];
                res = (res > 0.0) ? res : 0.0;
                if (nxt) nxt[v] = res;
                return res;
            }, false, nullptr);
            if (Z > 0.0 && n_rej < kMaxRejected) {
                if (tid == 0) { s_rej[n_rej] = c; s_Z[n_rej] = Z; }
                if (nxt) cur = (nxt == buf1) ? 1 : 0;
                inv_Z = 1.0 / Z;
                ++n_rej;
            }
            __syncthreads();
        }
        if (next >= 0) {
            if (tid == 0 && A < MIRROR_MAX_DEPTH) s_path[A] = next;
            ++A;
            r = next;
            __syncthreads();
            if (A >= MIRROR_MAX_DEPTH) { n_children = 0; n_rej = 0; break; }      // (cannot happen: depth <= gamma <= 32)
            continue;
        }
        break;
    }
    const bool have_extra = (n_children > 0) || a.emit_bonus != 0;
    if (tid == 0) { s_extra = -1; s_last = -1; s_found = -1; }
    __syncthreads();
    if (have_extra) {
        // inverse-CDF draw from m at row r: the CTA whose slice holds the crossing searches it
        const size_t row = (size_t)b * n + r;
        const float* lr = a.logits + row * V;
        const double lse_r = (double)a.lse[row];
        double excl_cta = 0.0;
        const double tot = cluster_total([&](int v) { return mass(lr, lse_r, v); }, true, &excl_cta);
        const double thr = (double)a.u_resample[row] * tot;
        if (warp == 0) {
            double lp = 0.0;
            for (int k = 0; k < 32; ++k) lp += s_seg[lane * 32 + k];
            double dummy;
            double run = excl_cta + warp_excl_scan(lp, lane, &dummy);
            int found = -1;
            double found_excl = 0.0;
            for (int k = 0; k < 32; ++k) {
                const double seg = s_seg[lane * 32 + k];
                if (found < 0 && run + seg > thr) { found = lane * 32 + k; found_excl = run; }
                run += seg;
            }
            // only the first CTA whose cumulative sum passes the threshold holds the crossing
            if (!(excl_cta <= thr)) found = -1;
            const unsigned mk = __ballot_sync(0xffffffffu, found >= 0);
            if (mk) {
                const int src = __ffs(mk) - 1;
                if (lane == src) { s_found = found; s_excl = found_excl; }
            }
        }
        __syncthreads();
        if (s_found >= 0 && tid == s_found) {
            const double excl = s_excl;
            double loc = 0.0;
            int pick = v1 - 1;
            for (int v = v0; v < v1; ++v) {
                loc += mass(lr, lse_r, v);
                if (excl + loc > thr) { pick = v; break; }
            }
            *cluster.map_shared_rank(&s_extra, 0) = pick;              // hand the token to the CTA that writes the outputs
        }
        cluster.sync();
        if (*cluster.map_shared_rank(&s_extra, 0) < 0) {
            // rounding left the threshold above every cumulative sum (the same in every CTA): the last id with positive mass
            int last = -1;
            for (int v = v0; v < v1; ++v)
                if (mass(lr, lse_r, v) > 0.0) last = v;
            if (last >= 0) atomicMax(&s_last, last);
            cluster.sync();
            if (rank == 0 && tid == 0) {
                int best_last = -1;
                for (int c = 0; c < kTreeCluster; ++c) best_last = max(best_last, *cluster.map_shared_rank(&s_last, c));
                s_extra = best_last;
            }
        }
    }
    __syncthreads();

    const int gamma = tp.gamma;
    if (rank == 0) {
        if (tid <= gamma) {
            int e = -1;
            if (tid < A) e = tok[s_path[tid]];
            else if (tid == A && have_extra) e = s_extra;
            a.out.emitted[(size_t)b * (gamma + 1) + tid] = e;
            if (tid < gamma) a.out.accepted_nodes[(size_t)b * gamma + tid] = (tid < A) ? s_path[tid] : -1;
        }
        if (tid == 0) {
            // the lowest-index branch that contains the accepted path
            int best = 0;
            for (int i = 0; i < tp.n_branches; ++i) {
                bool ok = tp.path_len[i] >= A;
                for (int k = 0; k < A && ok; ++k) ok = (tp.path[i][k] == s_path[k]);
                if (ok) { best = i; break; }
            }
            a.out.n_accepted[b] = A;
            a.out.best_branch[b] = best;
            a.out.decide_row[b] = r;
            a.out.n_emitted[b] = A + (have_extra ? 1 : 0);
            int slot = -1;
            if (have_extra && a.cand_ids)
                for (int k = 0; k < a.n_cand; ++k)
                    if (a.cand_ids[((size_t)b * n + r) * a.n_cand + k] == s_extra) { slot = k; break; }
            a.out.reuse_slot[b] = slot;
        }
    }
    // no CTA may leave while a peer can still read its shared memory
    cluster.sync();
}

}  // namespace

mirror_status mirror_accept_launch(mirror_ctx* ctx, const mirror_tree* tree, const MirrorTreeInfo& ti,
                                   const mirror_accept_in* in, const mirror_accept_out* out, cudaStream_t stream,
                                   double* tree_scratch) {
    AcceptTreeParams tp;
    tp.n = ti.n;
    tp.n_branches = ti.n_branches;
    tp.gamma = tree->gamma;
    for (int i = 0; i < MIRROR_MAX_NODES; ++i) tp.parent[i] = (i < ti.n && ti.parent[i] >= 0) ? (unsigned char)ti.parent[i] : 255;
    memcpy(tp.path, ti.path, sizeof tp.path);
    memcpy(tp.path_len, ti.path_len, sizeof tp.path_len);
    AcceptArgs a;
    a.mode = in->mode;
    a.emit_bonus = in->emit_bonus;
    a.V = ctx->desc.vocab;
    a.n_cand = in->cand_ids ? in->n_cand : 0;
    a.inv_T = 1.0 / (double)ctx->temperature;
    a.tokens = tree->tokens;
    a.target_argmax = in->target_argmax;
    a.logits = in->logits;
    a.lse = in->lse;
    a.q_probs = in->q_probs;
    a.u_accept = in->u_accept;
    a.u_resample = in->u_resample;
    a.cand_ids = in->cand_ids;
    a.out = *out;
    a.tree_scratch = tree_scratch;
    a.status = ctx->d_status;
    if (in->mode == MIRROR_ACCEPT_SPEC_TREE) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)tree->batch * kTreeCluster);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = stream;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = kTreeCluster;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        MIRROR_CUDA_OK(cudaLaunchKernelEx(&cfg, accept_tree_kernel, tp, a));
    } else MIRROR_CUDA_OK(mirror_launch_pdl(accept_select_kernel, dim3(tree->batch), dim3(kThreads), 0, stream, tp, a));
    ctx->launches += 1;
    MIRROR_CUDA_OK(cudaGetLastError());
    return MIRROR_OK;
}

extern "C" mirror_status mirror_accept_select(mirror_ctx* ctx, const mirror_tree* tree, const mirror_accept_in* in,
                                              const mirror_accept_out* out, void* stream) {
    if (!ctx || !tree || !in || !out || !tree->tokens) return MIRROR_ERR_ARG;
    if (!out->n_accepted || !out->best_branch || !out->n_emitted || !out->emitted || !out->accepted_nodes ||
        !out->decide_row || !out->reuse_slot)
        return MIRROR_ERR_ARG;
    if (in->mode == MIRROR_ACCEPT_GREEDY) {
        if (!in->target_argmax) return MIRROR_ERR_ARG;
    } else if (in->mode == MIRROR_ACCEPT_SPEC_SAMPLING || in->mode == MIRROR_ACCEPT_SPEC_TREE) {
        if (!in->logits || !in->lse || !in->u_accept || !in->u_resample) return MIRROR_ERR_ARG;
        if (tree->n_nodes > 1 && !in->q_probs) return MIRROR_ERR_ARG;
    } else {
        return MIRROR_ERR_ARG;
    }
    if (in->cand_ids && in->n_cand < 0) return MIRROR_ERR_ARG;
    MirrorTreeInfo ti;
    mirror_status st = mirror_build_tree(tree, &ti);
    if (st != MIRROR_OK) return st;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    double* tree_scratch = nullptr;
    if (in->mode == MIRROR_ACCEPT_SPEC_TREE && ctx->ws) {
        MirrorWsLayout L;
        mirror_ws_layout(ctx, (size_t)tree->batch * tree->n_nodes, &L, (size_t)tree->batch);
        if (ctx->ws_bytes >= L.end_accept) tree_scratch = (double*)((uint8_t*)ctx->ws + L.accept_scratch);
    }
    return mirror_accept_launch(ctx, tree, ti, in, out, (cudaStream_t)stream, tree_scratch);
}
