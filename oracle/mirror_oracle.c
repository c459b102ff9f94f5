/*
 * CPU oracle for the target-side verify step of Mirror Speculative Decoding.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow definition of what the
 * verify step computes; the parity tests, the smoke check and the benchmark's
 * cpu_baseline leg call it, nothing else does.  It shares no code with the CUDA
 * library and includes none of its headers.
 *
 * All floating-point work is fp64.  Tensors that the GPU path stores in bf16
 * (Q, K, V, hidden rows, LM-head weights) are taken here as their bf16 bit
 * patterns and widened exactly, so both sides start from identical values.
 *
 * There is no blocking, fusion or reordering: every function is the textbook
 * definition written out as loops (OpenMP only distributes independent output
 * elements over threads; no reduction is split across threads).
 *
 * Pins (tests/test_oracle_*.py): per-branch causal decoding by brute force, a
 * library attention routine with an explicit mask, softmax invariants, closed
 * forms for the LM head, exhaustive enumeration of the greedy rule, exact
 * integration of the speculative-sampling rule for one branch (losslessness),
 * the worked example of Fig. 1, and the reuse probability of Proposition 1.
 * The independent per-branch speculative-sampling rule over kappa > 1 branches
 * (oracle_accept_spec) is this build's own reading (the paper verifies one path
 * per step); for kappa > 1 it is pinned against that reading by hand-worked cases
 * with deterministic uniforms (ties and A = 0 go to the lowest branch, the longer
 * branch wins at any index, the residual and its uniform belong to the chosen
 * branch's deciding row and first rejected node).  The lossless rule over sibling sets
 * (oracle_accept_tree) is pinned by exact integration for two and three independent
 * siblings (the emitted token follows the target distribution), by its chain special
 * case (equal to the single-branch rule) and by fixed walk-order cases.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_f64(uint16_t bits) {
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ------------------------------------------------------------------------------------------
 * Hypothesis tree (Sec. 3.1, "hypothesis tree T_t"): node 0 is the last committed token,
 * parent[i] < i.  anc[i*n + j] = 1 iff j == i or j is an ancestor of i: the set of tree
 * tokens that node i may attend to.  Returns 0, or -1 for a malformed parent array.
 * ---------------------------------------------------------------------------------------- */
int oracle_tree(const int32_t* parent, int n, uint8_t* anc, int32_t* depth) {
    if (n < 1 || parent[0] != -1) return -1;
    memset(anc, 0, (size_t)n * n);
    for (int i = 0; i < n; ++i) {
        if (i > 0 && (parent[i] < 0 || parent[i] >= i)) return -1;
        int dpt = 0;
        for (int j = i; j != -1; j = parent[j]) {
            anc[(size_t)i * n + j] = 1;
            if (j != i) ++dpt;
        }
        depth[i] = dpt;
    }
    return 0;
}

/* Root-to-leaf paths ("branches").  Leaves are taken in increasing node order; path b lists
 * the non-root nodes from depth 1 down to the leaf, padded with -1 to max_len entries.
 * Returns the number of branches, or -1 if a path is longer than max_len. */
int oracle_branches(const int32_t* parent, int n, int max_len, int32_t* paths, int32_t* path_len) {
    int nb = 0;
    for (int leaf = 1; leaf < n; ++leaf) {
        int is_leaf = 1;
        for (int c = leaf + 1; c < n; ++c)
            if (parent[c] == leaf) { is_leaf = 0; break; }
        if (!is_leaf) continue;
        int len = 0;
        for (int j = leaf; j != 0; j = parent[j]) ++len;
        if (len > max_len) return -1;
        for (int k = 0; k < max_len; ++k) paths[(size_t)nb * max_len + k] = -1;
        int pos = len - 1;
        for (int j = leaf; j != 0; j = parent[j]) paths[(size_t)nb * max_len + pos--] = j;
        path_len[nb] = len;
        ++nb;
    }
    return nb;
}

/* ------------------------------------------------------------------------------------------
 * O1. Branch-tree attention of one layer (the attention inside the target forward whose
 * last state feeds Softmax(W h), Eq. 1; the tree mask restricts node i to the verified prefix
 * plus its own root-to-node path, so that every branch is scored exactly as if it were decoded
 * alone, which is what "verifies left-to-right" in Eq. 3 requires).
 *
 *   Vis(i)  = { prefix token t : 0 <= t < L_b }  U  { tree token j : anc[i][j] }
 *   s_t     = scale * <q_i,h , k_t,g>            g = h / (Hq/Hkv)
 *   w       = softmax over Vis(i)
 *   o_i,h   = sum_t w_t v_t,g
 *
 * Layouts: q [B,n,Hq,d]; pools [num_pages,Hkv,P,d]; k_new/v_new [B,n,Hkv,d];
 * page_table [B,max_pages]; out [B,n,Hq,d]; lse [B,Hq,n] (natural log of the softmax
 * denominator, shifted back: log sum exp s); weights (optional) [B,n,Hq,Lmax+n] holds every
 * softmax weight, zeros where masked (Lmax = max_pages*P), for invariant checks.
 * ---------------------------------------------------------------------------------------- */
void oracle_attention_layer(const uint16_t* q, const uint16_t* k_pool, const uint16_t* v_pool,
                            const int32_t* page_table, int max_pages, const int32_t* prefix_len,
                            const uint16_t* k_new, const uint16_t* v_new, const uint8_t* anc,
                            int B, int n, int Hq, int Hkv, int d, int P, double scale,
                            double* out, double* lse, double* weights) {
    const int G = Hq / Hkv;
    const int Lmax = max_pages * P;
#pragma omp parallel for collapse(3) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < n; ++i)
            for (int h = 0; h < Hq; ++h) {
                const int g = h / G;
                const int L = prefix_len[b];
                const uint16_t* qv = q + (((size_t)b * n + i) * Hq + h) * d;
                double* s = (double*)malloc(sizeof(double) * (size_t)(L + n));
                /* scores over the visible set; masked tree tokens are simply absent */
                double m = -INFINITY;
                for (int t = 0; t < L + n; ++t) {
                    const uint16_t* kv;
                    if (t < L) {
                        int page = page_table[(size_t)b * max_pages + t / P];
                        kv = k_pool + (((size_t)page * Hkv + g) * P + t % P) * d;
                    } else {
                        int j = t - L;
                        if (!anc[(size_t)i * n + j]) { s[t] = -INFINITY; continue; }
                        kv = k_new + (((size_t)b * n + j) * Hkv + g) * d;
                    }
                    double acc = 0.0;
                    for (int e = 0; e < d; ++e) acc += bf16_to_f64(qv[e]) * bf16_to_f64(kv[e]);
                    s[t] = scale * acc;
                    if (s[t] > m) m = s[t];
                }
                double denom = 0.0;
                for (int t = 0; t < L + n; ++t)
                    if (s[t] != -INFINITY) denom += exp(s[t] - m);
                double* o = out + (((size_t)b * n + i) * Hq + h) * d;
                for (int e = 0; e < d; ++e) o[e] = 0.0;
                for (int t = 0; t < L + n; ++t) {
                    double w = (s[t] == -INFINITY) ? 0.0 : exp(s[t] - m) / denom;
                    if (weights) {
                        size_t col = (t < L) ? (size_t)t : (size_t)Lmax + (t - L);
                        weights[(((size_t)b * n + i) * Hq + h) * (size_t)(Lmax + n) + col] = w;
                    }
                    if (w == 0.0) continue;
                    const uint16_t* vv;
                    if (t < L) {
                        int page = page_table[(size_t)b * max_pages + t / P];
                        vv = v_pool + (((size_t)page * Hkv + g) * P + t % P) * d;
                    } else {
                        vv = v_new + (((size_t)b * n + (t - L)) * Hkv + g) * d;
                    }
                    for (int e = 0; e < d; ++e) o[e] += w * bf16_to_f64(vv[e]);
                }
                if (lse) lse[((size_t)b * Hq + h) * n + i] = m + log(denom);
                free(s);
            }
}

/* ------------------------------------------------------------------------------------------
 * O2. LM head (Eq. 1: the distribution is Softmax(W h), W in R^{|V| x H}; the same map
 * applied to an intermediate state gives the early-exit proxy, Eq. 5):
 *     logits[r][v] = sum_k hidden[r][k] * W[v][k]
 * ---------------------------------------------------------------------------------------- */
void oracle_lmhead_logits(const uint16_t* hidden, const uint16_t* W, int M, int V, int H, double* logits) {
#pragma omp parallel for schedule(static)
    for (int v = 0; v < V; ++v)
        for (int r = 0; r < M; ++r) {
            double acc = 0.0;
            for (int k = 0; k < H; ++k)
                acc += bf16_to_f64(hidden[(size_t)r * H + k]) * bf16_to_f64(W[(size_t)v * H + k]);
            logits[(size_t)r * V + v] = acc;
        }
}

/* Same, for rows whose hidden state is already fp64 (the chained step feeds attention output). */
void oracle_lmhead_logits_f64(const double* hidden, const uint16_t* W, int M, int V, int H, double* logits) {
#pragma omp parallel for schedule(static)
    for (int v = 0; v < V; ++v)
        for (int r = 0; r < M; ++r) {
            double acc = 0.0;
            for (int k = 0; k < H; ++k) acc += hidden[(size_t)r * H + k] * bf16_to_f64(W[(size_t)v * H + k]);
            logits[(size_t)r * V + v] = acc;
        }
}

/* Row reductions of the logits: the argmax that greedy verification compares against (Eq. 3),
 * the log-normaliser of Softmax(logits / T), and the Top-kappa message of Eq. 6: ids with their
 * log-probabilities.  Order everywhere: logit descending, then token id ascending, so ties go to
 * the lowest id.  topk_id/topk_logprob are [M,topk] (ignored when topk == 0). */
void oracle_row_reduce(const double* logits, int M, int V, double temperature, int topk,
                       int32_t* argmax, double* maxlogit, double* lse,
                       int32_t* topk_id, double* topk_logprob) {
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < M; ++r) {
        const double* l = logits + (size_t)r * V;
        int best = 0;
        for (int v = 1; v < V; ++v)
            if (l[v] > l[best]) best = v;      /* strict: the first (lowest) id keeps a tie */
        double m = l[best] / temperature, sum = 0.0;
        for (int v = 0; v < V; ++v) sum += exp(l[v] / temperature - m);
        double row_lse = m + log(sum);
        if (argmax) argmax[r] = best;
        if (maxlogit) maxlogit[r] = l[best];
        if (lse) lse[r] = row_lse;
        for (int k = 0; k < topk; ++k) {
            /* k-th element of the order: the best id not already taken */
            int pick = -1;
            for (int v = 0; v < V; ++v) {
                int taken = 0;
                for (int j = 0; j < k; ++j)
                    if (topk_id[(size_t)r * topk + j] == v) { taken = 1; break; }
                if (taken) continue;
                if (pick < 0 || l[v] > l[pick]) pick = v;
            }
            topk_id[(size_t)r * topk + k] = pick;
            topk_logprob[(size_t)r * topk + k] = l[pick] / temperature - row_lse;
        }
    }
}

/* ------------------------------------------------------------------------------------------
 * O3. Greedy acceptance, branch selection and reuse lookup.
 *
 * Per branch (root-to-leaf path c_1..c_len) the accepted length is the acceptance operator
 * of Eq. 3 / Eq. 10:  a = max{ r : tok[c_j] == argmax[parent(c_j)]  for all j <= r }
 * (the row of a node's parent is the target distribution that node's token is checked
 * against: left-to-right, teacher-forced).  A = max over branches; the chosen branch is the
 * lowest-index branch attaining it.  The deciding row R is the last accepted node (the root if
 * A == 0); the correction token (A < len) or bonus token (A == len) is argmax[R].
 * Reuse (Sec. 3.1, "Verification vs. reuse criterion"): the corrected prefix is already in the
 * hypothesis tree iff the correction token is among the candidates recorded for row R;
 * reuse_slot is its index in cand_ids[b][R][:], else -1 (fallback: fresh rollout).
 *
 * tokens, target_argmax: [B,n]; cand_ids: [B,n,n_cand] or NULL.
 * Outputs per request: n_accepted, best_branch, decide_row, n_emitted, reuse_slot: [B];
 * emitted: [B,max_len+1] (-1 padded); accepted_nodes: [B,max_len] (-1 padded).
 * Returns 0, -1 for a bad tree.
 * ---------------------------------------------------------------------------------------- */
int oracle_accept_greedy(const int32_t* tokens, const int32_t* target_argmax, const int32_t* parent,
                         int B, int n, int max_len, int emit_bonus,
                         const int32_t* cand_ids, int n_cand,
                         int32_t* n_accepted, int32_t* best_branch, int32_t* decide_row,
                         int32_t* n_emitted, int32_t* emitted, int32_t* accepted_nodes,
                         int32_t* reuse_slot) {
    int32_t* paths = (int32_t*)malloc(sizeof(int32_t) * (size_t)n * max_len);
    int32_t* plen = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    int nb = oracle_branches(parent, n, max_len, paths, plen);
    if (nb < 0) { free(paths); free(plen); return -1; }
    for (int b = 0; b < B; ++b) {
        const int32_t* tok = tokens + (size_t)b * n;
        const int32_t* am = target_argmax + (size_t)b * n;
        int A = 0, best = 0;
        for (int i = 0; i < nb; ++i) {
            int a = 0;
            while (a < plen[i]) {
                int c = paths[(size_t)i * max_len + a];
                if (tok[c] != am[parent[c]]) break;
                ++a;
            }
            if (a > A) { A = a; best = i; }     /* strict: lowest branch index keeps a tie */
        }
        int R = (A == 0) ? 0 : paths[(size_t)best * max_len + A - 1];
        for (int k = 0; k < max_len + 1; ++k) emitted[(size_t)b * (max_len + 1) + k] = -1;
        for (int k = 0; k < max_len; ++k) accepted_nodes[(size_t)b * max_len + k] = -1;
        for (int k = 0; k < A; ++k) {
            int c = paths[(size_t)best * max_len + k];
            accepted_nodes[(size_t)b * max_len + k] = c;
            emitted[(size_t)b * (max_len + 1) + k] = tok[c];
        }
        int have_extra = (nb == 0 || A < plen[best]) ? 1 : (emit_bonus != 0);
        int extra = am[R];
        int ne = A;
        if (have_extra) emitted[(size_t)b * (max_len + 1) + ne++] = extra;
        n_accepted[b] = A; best_branch[b] = best; decide_row[b] = R; n_emitted[b] = ne;
        int slot = -1;
        if (have_extra && cand_ids)
            for (int k = 0; k < n_cand; ++k)
                if (cand_ids[((size_t)b * n + R) * n_cand + k] == extra) { slot = k; break; }
        reuse_slot[b] = slot;
    }
    free(paths); free(plen);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * O3'. Speculative-sampling acceptance ("the standard speculative rule", Sec. 3.1, of the works
 * the paper builds on: accept a drafted token x with probability min(1, p(x)/q(x)); on the first
 * rejection draw the correction from the normalised residual max(0, p - q); if the whole window
 * is accepted draw a bonus token from p).
 *
 * With p_r = Softmax(logits[r] / T) taken as  p_r[v] = exp(logits[r][v]/T - lse[r])  where lse
 * is the GIVEN log-normaliser of row r (the LM-head reduction's output), node c with token x,
 * parent row r and draft distribution q_c is accepted iff   u_accept[c] * q_c[x] <= p_r[x].
 * Branch lengths, A, the chosen branch and the deciding row R are as in the greedy rule.
 * Extra token at R with uniform u = u_resample[R]:
 *   A < len: c' = first rejected node of the chosen branch; res_v = max(0, p_R[v] - q_c'[v]);
 *            Z = sum_v res_v; token = min{ v : sum_{w<=v} res_w > u*Z };  Z == 0 falls back to p_R.
 *   A == len: the same inverse-CDF draw from p_R itself.
 * If rounding leaves no v beyond the threshold, the last id with positive mass is returned.
 * Sums run in increasing id order.  margin[b] receives the smallest relative distance to a
 * decision boundary seen while deciding request b (accept tests and the CDF crossing), so that
 * a caller comparing against another implementation can tell a knife-edge from a real mismatch.
 *
 * logits [B*n,V] fp32, lse [B*n] fp32, q_probs [B,n-1,V] fp32 (row c-1 is node c's draft
 * distribution), u_accept/u_resample [B,n] fp32.
 * ---------------------------------------------------------------------------------------- */
static int inverse_cdf(const double* mass, int V, double u, double* margin) {
    double Z = 0.0;
    for (int v = 0; v < V; ++v) Z += mass[v];
    double thr = u * Z, run = 0.0;
    int last_pos = -1;
    for (int v = 0; v < V; ++v) {
        if (mass[v] > 0.0) last_pos = v;
        double prev = run;
        run += mass[v];
        if (run > thr) {
            double rel = fmin(run - thr, thr - prev) / (Z > 0 ? Z : 1.0);
            if (rel < *margin) *margin = rel;
            return v;
        }
    }
    *margin = 0.0;
    return last_pos;
}

int oracle_accept_spec(const int32_t* tokens, const float* logits, const float* lse, const float* q_probs,
                       const float* u_accept, const float* u_resample, const int32_t* parent,
                       int B, int n, int V, int max_len, int emit_bonus, double temperature,
                       const int32_t* cand_ids, int n_cand,
                       int32_t* n_accepted, int32_t* best_branch, int32_t* decide_row,
                       int32_t* n_emitted, int32_t* emitted, int32_t* accepted_nodes,
                       int32_t* reuse_slot, double* margin) {
    int32_t* paths = (int32_t*)malloc(sizeof(int32_t) * (size_t)n * max_len);
    int32_t* plen = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    int nb = oracle_branches(parent, n, max_len, paths, plen);
    if (nb < 0) { free(paths); free(plen); return -1; }
    double* mass = (double*)malloc(sizeof(double) * (size_t)V);
    for (int b = 0; b < B; ++b) {
        const int32_t* tok = tokens + (size_t)b * n;
        double mg = INFINITY;
        int A = 0, best = 0;
        for (int i = 0; i < nb; ++i) {
            int a = 0;
            while (a < plen[i]) {
                int c = paths[(size_t)i * max_len + a];
                int r = parent[c], x = tok[c];
                size_t row = (size_t)b * n + r;
                double p = exp((double)logits[row * V + x] / temperature - (double)lse[row]);
                double lhs = (double)u_accept[(size_t)b * n + c] *
                             (double)q_probs[((size_t)b * (n - 1) + (c - 1)) * V + x];
                double rel = fabs(lhs - p) / (p > 0 ? p : 1.0);
                if (rel < mg) mg = rel;
                if (!(lhs <= p)) break;
                ++a;
            }
            if (a > A) { A = a; best = i; }
        }
        int R = (A == 0) ? 0 : paths[(size_t)best * max_len + A - 1];
        size_t rowR = (size_t)b * n + R;
        for (int k = 0; k < max_len + 1; ++k) emitted[(size_t)b * (max_len + 1) + k] = -1;
        for (int k = 0; k < max_len; ++k) accepted_nodes[(size_t)b * max_len + k] = -1;
        for (int k = 0; k < A; ++k) {
            int c = paths[(size_t)best * max_len + k];
            accepted_nodes[(size_t)b * max_len + k] = c;
            emitted[(size_t)b * (max_len + 1) + k] = tok[c];
        }
        int rejected = (nb > 0 && A < plen[best]);
        int have_extra = rejected || nb == 0 || emit_bonus != 0;
        int ne = A, extra = -1;
        if (have_extra) {
            double u = (double)u_resample[(size_t)b * n + R];
            for (int v = 0; v < V; ++v)
                mass[v] = exp((double)logits[rowR * V + v] / temperature - (double)lse[rowR]);
            if (rejected) {
                int cr = paths[(size_t)best * max_len + A];
                const float* qc = q_probs + ((size_t)b * (n - 1) + (cr - 1)) * V;
                double Z = 0.0;
                for (int v = 0; v < V; ++v) {
                    double res = mass[v] - (double)qc[v];
                    Z += (res > 0.0) ? res : 0.0;
                }
                if (Z > 0.0)
                    for (int v = 0; v < V; ++v) {
                        double res = mass[v] - (double)qc[v];
                        mass[v] = (res > 0.0) ? res : 0.0;
                    }
            }
            extra = inverse_cdf(mass, V, u, &mg);
            emitted[(size_t)b * (max_len + 1) + ne++] = extra;
        }
        n_accepted[b] = A; best_branch[b] = best; decide_row[b] = R; n_emitted[b] = ne;
        int slot = -1;
        if (have_extra && cand_ids)
            for (int k = 0; k < n_cand; ++k)
                if (cand_ids[((size_t)b * n + R) * n_cand + k] == extra) { slot = k; break; }
        reuse_slot[b] = slot;
        if (margin) margin[b] = mg;
    }
    free(mass); free(paths); free(plen);
    return 0;
}

/* ----------------------------------------------------------------------------------------
 * O3'': lossless acceptance over a token tree (Sec. 3.1's speculative-sampling rule applied to the
 * sibling sets of a tree draft: sequential multi-round rejection).
 * Walk down from the root.  At row r the target distribution is p_r; its children c_1 < c_2 < ...
 * (node order) are tested one after the other against the CURRENT distribution m (m = p_r at first):
 * child c with token x and draft distribution q_c passes iff u_accept[c] * q_c[x] <= m[x]; the walk
 * then moves to row c.  A child that fails turns m into the normalised residual max(0, m - q_c)
 * (left unchanged when that residual has no mass).  When every child of r has failed, or r is a
 * leaf and emit_bonus is set, the extra token is drawn from m by inverse CDF with u_resample[r].
 * If the siblings of a node are independent draws from one q, the emitted tokens are distributed
 * exactly as the target's own samples, for any number of siblings.
 * best_branch is the lowest-index root-to-leaf branch that contains the accepted path.
 * margin[b]: smallest relative distance of any decision of request b from its knife edge.
 * ---------------------------------------------------------------------------------------- */
int oracle_accept_tree(const int32_t* tokens, const float* logits, const float* lse, const float* q_probs,
                       const float* u_accept, const float* u_resample, const int32_t* parent,
                       int B, int n, int V, int max_len, int emit_bonus, double temperature,
                       const int32_t* cand_ids, int n_cand,
                       int32_t* n_accepted, int32_t* best_branch, int32_t* decide_row,
                       int32_t* n_emitted, int32_t* emitted, int32_t* accepted_nodes,
                       int32_t* reuse_slot, double* margin) {
    int32_t* paths = (int32_t*)malloc(sizeof(int32_t) * (size_t)n * max_len);
    int32_t* plen = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    int nb = oracle_branches(parent, n, max_len, paths, plen);
    if (nb < 0) { free(paths); free(plen); return -1; }
    double* m = (double*)malloc(sizeof(double) * (size_t)V);
    for (int b = 0; b < B; ++b) {
        const int32_t* tok = tokens + (size_t)b * n;
        double mg = INFINITY;
        for (int k = 0; k < max_len + 1; ++k) emitted[(size_t)b * (max_len + 1) + k] = -1;
        for (int k = 0; k < max_len; ++k) accepted_nodes[(size_t)b * max_len + k] = -1;
        int r = 0, A = 0, ne = 0, extra = -1, have_extra = 0;
        for (;;) {
            size_t row = (size_t)b * n + r;
            for (int v = 0; v < V; ++v) m[v] = exp((double)logits[row * V + v] / temperature - (double)lse[row]);
            int n_children = 0, next = -1;
            for (int c = r + 1; c < n && next < 0; ++c) {
                if (parent[c] != r) continue;
                ++n_children;
                int x = tok[c];
                const float* qc = q_probs + ((size_t)b * (n - 1) + (c - 1)) * V;
                double lhs = (double)u_accept[(size_t)b * n + c] * (double)qc[x];
                double rel = fabs(lhs - m[x]) / (m[x] > 0 ? m[x] : 1.0);
                if (rel < mg) mg = rel;
                if (lhs <= m[x]) { next = c; break; }
                double Z = 0.0;
                for (int v = 0; v < V; ++v) {
                    double res = m[v] - (double)qc[v];
                    Z += (res > 0.0) ? res : 0.0;
                }
                if (Z > 0.0)
                    for (int v = 0; v < V; ++v) {
                        double res = m[v] - (double)qc[v];
                        m[v] = ((res > 0.0) ? res : 0.0) / Z;
                    }
            }
            if (next >= 0) {
                accepted_nodes[(size_t)b * max_len + A] = next;
                emitted[(size_t)b * (max_len + 1) + A] = tok[next];
                ++A;
                r = next;
                continue;
            }
            have_extra = (n_children > 0) || emit_bonus != 0;
            if (have_extra) extra = inverse_cdf(m, V, (double)u_resample[(size_t)b * n + r], &mg);
            break;
        }
        ne = A;
        if (have_extra) emitted[(size_t)b * (max_len + 1) + ne++] = extra;
        int best = 0;
        for (int i = 0; i < nb; ++i) {
            int ok = plen[i] >= A;
            for (int k = 0; k < A && ok; ++k) ok = paths[(size_t)i * max_len + k] == accepted_nodes[(size_t)b * max_len + k];
            if (ok) { best = i; break; }
        }
        n_accepted[b] = A; best_branch[b] = best; decide_row[b] = r; n_emitted[b] = ne;
        int slot = -1;
        if (have_extra && cand_ids)
            for (int k = 0; k < n_cand; ++k)
                if (cand_ids[((size_t)b * n + r) * n_cand + k] == extra) { slot = k; break; }
        reuse_slot[b] = slot;
        if (margin) margin[b] = mg;
    }
    free(m); free(paths); free(plen);
    return 0;
}

/* Overlap mass of Eq. 7: Omega_kappa = sum of the final distribution q over the early-exit
 * Top-kappa ids.  q_final [V] probabilities, ids [kappa]. */
double oracle_overlap_mass(const double* q_final, const int32_t* ids, int kappa) {
    double s = 0.0;
    for (int k = 0; k < kappa; ++k) s += q_final[ids[k]];
    return s;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
