// Acceptance, branch selection, emitted tokens and reuse lookup (Sec. 3.1; Eq. 3 / Eq. 10).
//
// One thread block per request.  Warps take branches round-robin; lane j of a warp tests the node at
// depth j+1 of its branch, a ballot gives the number of leading passes (the acceptance operator of
// Eq. 3 applied to that branch).  Thread 0 then picks the longest branch (lowest index on ties) and the
// deciding row R.  Greedy mode emits argmax[R]; speculative-sampling mode draws the extra token by an
// inverse-CDF search over the vocabulary that the whole block cooperates on, all in fp64.
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
                atomicExch(a.status, MIRROR_DEV_CHECK);
                atomicExch(a.status + 1, 100 + c);
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

}  // namespace

mirror_status mirror_accept_launch(mirror_ctx* ctx, const mirror_tree* tree, const MirrorTreeInfo& ti,
                                   const mirror_accept_in* in, const mirror_accept_out* out, cudaStream_t stream) {
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
    a.status = ctx->d_status;
    accept_select_kernel<<<tree->batch, kThreads, 0, stream>>>(tp, a);
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
    } else if (in->mode == MIRROR_ACCEPT_SPEC_SAMPLING) {
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
    return mirror_accept_launch(ctx, tree, ti, in, out, (cudaStream_t)stream);
}
