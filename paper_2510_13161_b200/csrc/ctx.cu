// Context, argument digests (token tree), workspace carving, tensor maps, status plumbing.
#include <stdlib.h>
#include <string.h>

#include <new>

#include "mirror_internal.h"

extern "C" const char* mirror_status_str(mirror_status s) {
    switch (s) {
        case MIRROR_OK: return "ok";
        case MIRROR_ERR_ARG: return "bad argument (null pointer or negative size)";
        case MIRROR_ERR_SHAPE: return "inconsistent or out-of-range dimensions";
        case MIRROR_ERR_UNSUPPORTED: return "unsupported configuration or device";
        case MIRROR_ERR_WORKSPACE: return "workspace missing or too small";
        case MIRROR_ERR_CUDA: return "CUDA call failed";
        case MIRROR_ERR_DEVICE_CHECK: return "device-side bounds check tripped";
        case MIRROR_ERR_TIMEOUT: return "bounded device-side wait expired";
    }
    return "unknown status";
}

extern "C" mirror_status mirror_create(mirror_ctx** out, const mirror_model_desc* desc, int device) {
    if (!out || !desc) return MIRROR_ERR_ARG;
    *out = nullptr;
    if (desc->hidden <= 0 || desc->n_q_heads <= 0 || desc->n_kv_heads <= 0 || desc->vocab <= 0) return MIRROR_ERR_ARG;
    if (desc->n_q_heads % desc->n_kv_heads != 0) return MIRROR_ERR_SHAPE;
    if (desc->hidden % 64 != 0) return MIRROR_ERR_SHAPE;
    if (desc->head_dim != 64 && desc->head_dim != 128) return MIRROR_ERR_UNSUPPORTED;
    if (desc->page_size != 16) return MIRROR_ERR_UNSUPPORTED;
    if (desc->temperature < 0.f || desc->softmax_scale < 0.f) return MIRROR_ERR_ARG;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return MIRROR_ERR_CUDA;
    MIRROR_CUDA_OK(cudaSetDevice(device));
    cudaDeviceProp prop;
    MIRROR_CUDA_OK(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return MIRROR_ERR_UNSUPPORTED;   // the kernels are sm_100a only: no fallback path

    mirror_ctx* ctx = new (std::nothrow) mirror_ctx();
    if (!ctx) return MIRROR_ERR_ARG;
    ctx->desc = *desc;
    mirror_tuning_from_env(&ctx->tune);
    ctx->device = device;
    ctx->num_sms = prop.multiProcessorCount;
    ctx->scale = desc->softmax_scale > 0.f ? desc->softmax_scale : 1.0f / sqrtf((float)desc->head_dim);
    ctx->temperature = desc->temperature > 0.f ? desc->temperature : 1.0f;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) {
        delete ctx;
        return MIRROR_ERR_CUDA;
    }
    ctx->encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    if (cudaMalloc(&ctx->d_status, 2 * sizeof(int)) != cudaSuccess || cudaMemset(ctx->d_status, 0, 2 * sizeof(int)) != cudaSuccess) {
        delete ctx;
        return MIRROR_ERR_CUDA;
    }
    *out = ctx;
    return MIRROR_OK;
}

void mirror_tuning_from_env(MirrorTuning* t) {
    auto geti = [](const char* name, int* v, int lo, int hi) {
        if (const char* e = getenv(name)) { const long x = strtol(e, nullptr, 10); if (x >= lo && x <= hi) *v = (int)x; }
    };
    geti("MIRROR_ATTN_GROUPS", &t->attn_groups, 1, 1 << 20);
    geti("MIRROR_ATTN_WHOLE_UNITS", &t->attn_whole_units, 0, 1);
    geti("MIRROR_ATTN_SNAP", &t->attn_snap, 0, 1 << 20);
    geti("MIRROR_ATTN_RING", &t->attn_ring, 44, 66);
    geti("MIRROR_LM_PAIR2_MAX_ROWS", &t->lm_pair2_max_rows, 0, 128);
    geti("MIRROR_LM_CTAS_PER_SM", &t->lm_ctas_per_sm, 1, 2);
    geti("MIRROR_LM_STAGES", &t->lm_stages, 2, 64);
    geti("MIRROR_LM_ROWS", &t->lm_rows, 8, 128);
    geti("MIRROR_LM_PAIR_MIN_ROWS", &t->lm_pair_min_rows, 0, 1 << 30);
    geti("MIRROR_LM_KGROUP", &t->lm_kgroup, 1, 64);
    geti("MIRROR_TEST_STALL_AFTER_STAGES", &t->test_stall_after, 0, 1 << 30);
    if (const char* e = getenv("MIRROR_WAIT_LIMIT_CYCLES")) { const long long x = strtoll(e, nullptr, 10); if (x >= 1000) t->wait_limit_cycles = x; }
}

extern "C" mirror_status mirror_destroy(mirror_ctx* ctx) {
    if (!ctx) return MIRROR_ERR_ARG;
    cudaSetDevice(ctx->device);
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->copy_stream) {
        cudaStreamDestroy(ctx->copy_stream);
        for (cudaEvent_t e : ctx->copy_ev)
            if (e) cudaEventDestroy(e);
    }
    delete ctx;
    return MIRROR_OK;
}

extern "C" mirror_status mirror_device_status(mirror_ctx* ctx, int* code, int* detail) {
    if (!ctx || !code) return MIRROR_ERR_ARG;
    int h[2] = {0, 0};
    MIRROR_CUDA_OK(cudaDeviceSynchronize());
    MIRROR_CUDA_OK(cudaMemcpy(h, ctx->d_status, sizeof h, cudaMemcpyDeviceToHost));
    *code = h[0];
    if (detail) *detail = h[1];
    if (h[0] != 0) {
        MIRROR_CUDA_OK(cudaMemset(ctx->d_status, 0, sizeof h));
        if (ctx->ws) MIRROR_CUDA_OK(cudaMemset(ctx->ws, 0, ctx->ws_bytes < kWsZeroedBytes ? ctx->ws_bytes : kWsZeroedBytes));
    }
    return MIRROR_OK;
}

extern "C" mirror_status mirror_launch_count(const mirror_ctx* ctx, long long* count) {
    if (!ctx || !count) return MIRROR_ERR_ARG;
    *count = ctx->launches;
    return MIRROR_OK;
}

// ---------------------------------------------------------------------------------------------
// token tree digest
// ---------------------------------------------------------------------------------------------
mirror_status mirror_build_tree(const mirror_tree* tree, MirrorTreeInfo* info) {
    if (!tree || !info) return MIRROR_ERR_ARG;
    const int n = tree->n_nodes;
    if (tree->batch <= 0 || n <= 0 || tree->gamma < 0) return MIRROR_ERR_ARG;
    if (n > MIRROR_MAX_NODES || tree->gamma > MIRROR_MAX_DEPTH) return MIRROR_ERR_SHAPE;
    info->n = n;
    if (tree->parent) {
        if (tree->parent[0] != -1) return MIRROR_ERR_SHAPE;
        for (int i = 1; i < n; ++i)
            if (tree->parent[i] < 0 || tree->parent[i] >= i) return MIRROR_ERR_SHAPE;
        for (int i = 0; i < n; ++i) info->parent[i] = tree->parent[i];
    } else {
        if (tree->kappa < 0 || n != 1 + tree->kappa * tree->gamma) return MIRROR_ERR_SHAPE;
        info->parent[0] = -1;
        for (int i = 0; i < tree->kappa; ++i)
            for (int j = 0; j < tree->gamma; ++j) info->parent[1 + i * tree->gamma + j] = (j == 0) ? 0 : i * tree->gamma + j;
    }
    bool has_child[MIRROR_MAX_NODES] = {};
    for (int i = 0; i < n; ++i) {
        info->anc[i][0] = info->anc[i][1] = 0ull;
        int dpt = 0;
        for (int j = i; j != -1; j = info->parent[j]) {
            info->anc[i][j >> 6] |= 1ull << (j & 63);
            if (j != i) ++dpt;
        }
        info->depth[i] = dpt;
        if (dpt > tree->gamma) return MIRROR_ERR_SHAPE;
        if (i > 0) has_child[info->parent[i]] = true;
    }
    int nb = 0, max_len = 0;
    for (int leaf = 1; leaf < n; ++leaf) {
        if (has_child[leaf]) continue;
        if (nb >= MIRROR_MAX_BRANCHES) return MIRROR_ERR_SHAPE;
        const int len = info->depth[leaf];
        int pos = len - 1;
        for (int j = leaf; j != 0; j = info->parent[j]) info->path[nb][pos--] = (unsigned char)j;
        for (int k = len; k < MIRROR_MAX_DEPTH; ++k) info->path[nb][k] = 0;
        info->path_len[nb] = (unsigned char)len;
        if (len > max_len) max_len = len;
        ++nb;
    }
    info->n_branches = nb;
    info->max_len = max_len;
    return MIRROR_OK;
}

// ---------------------------------------------------------------------------------------------
// de-duplicated tree out of kappa branches (host only)
// ---------------------------------------------------------------------------------------------
extern "C" mirror_status mirror_trie_build(const int32_t* branch_tokens, int kappa, int gamma, int32_t root_token,
                                           int32_t* parent, int32_t* tokens, int32_t* node_of, int* n_nodes) {
    if (!branch_tokens || !parent || !tokens || !node_of || !n_nodes) return MIRROR_ERR_ARG;
    if (kappa <= 0 || gamma <= 0) return MIRROR_ERR_ARG;
    if (gamma > MIRROR_MAX_DEPTH || kappa > MIRROR_MAX_BRANCHES) return MIRROR_ERR_SHAPE;
    int n = 1;
    parent[0] = -1;
    tokens[0] = root_token;
    for (int i = 0; i < kappa; ++i) {
        int cur = 0;                                        // walk down from the root, growing the tree where needed
        for (int j = 0; j < gamma; ++j) {
            const int32_t t = branch_tokens[(size_t)i * gamma + j];
            int child = -1;
            for (int c = cur + 1; c < n; ++c)               // children always have larger ids than their parent
                if (parent[c] == cur && tokens[c] == t) { child = c; break; }
            if (child < 0) {
                if (n >= MIRROR_MAX_NODES) return MIRROR_ERR_SHAPE;
                child = n++;
                parent[child] = cur;
                tokens[child] = t;
            }
            node_of[(size_t)i * gamma + j] = child;
            cur = child;
        }
    }
    *n_nodes = n;
    return MIRROR_OK;
}

// ---------------------------------------------------------------------------------------------
// workspace
// ---------------------------------------------------------------------------------------------
void mirror_ws_layout(const mirror_ctx* ctx, size_t M, MirrorWsLayout* out, size_t B) {
    MirrorWsLayout L;
    size_t at = 0;
    L.zeroed = at;
    at += kWsZeroedBytes;
    L.attn_partial = at;
    // two partial slots per CTA (a CTA's range of KV tiles cuts at most two units), 128 rows each
    L.attn_partial_bytes = align_up((size_t)ctx->num_sms * 2 * 128 * (size_t)(ctx->desc.head_dim + 4) * sizeof(float), 256);
    at += L.attn_partial_bytes;
    L.end_attn = at;
    L.lm_partial = at;
    // one partial per CTA (up to two CTAs per SM) or per 128-row vocabulary tile (several row chunks), whichever is more
    const size_t per_cta = (size_t)2 * ctx->num_sms, per_tile = (size_t)mirror_lmhead_pair_partials(ctx->desc.vocab);
    const size_t n_part = per_cta > per_tile ? per_cta : per_tile;
    L.lm_partial_bytes = align_up(n_part * M * 12, 256);
    at += L.lm_partial_bytes;
    L.lse = at;
    at += align_up(M * sizeof(float), 256);
    L.argmax = at;
    at += align_up(M * sizeof(int), 256);
    L.end_lmhead = at;
    L.logits = at;
    L.logits_bytes = align_up(M * (size_t)ctx->desc.vocab * sizeof(float), 256);
    at += L.logits_bytes;
    L.end_logits = at;
    L.accept_scratch = at;
    at += align_up(B * 2 * (size_t)ctx->desc.vocab * sizeof(double), 256);
    L.end_accept = at;
    // the candidate lists of the fused Top-kappa share the front of the logits region (a call either spills or selects)
    L.lm_topk = L.logits;
    // (four lists per CTA and row, two CTAs per SM; only up to 256 rows, one row chunk: beyond, Top-kappa selects from spilled logits)
    L.lm_topk_bytes = M <= 256 ? align_up((size_t)8 * ctx->num_sms * M * (size_t)MIRROR_MAX_TOPK * 8, 256) : 0;
    L.end_topk = L.lm_topk + L.lm_topk_bytes;
    *out = L;
}

extern "C" mirror_status mirror_workspace_bytes(const mirror_ctx* ctx, const mirror_tree* tree, const mirror_kv* kv,
                                                unsigned what, size_t* bytes) {
    (void)kv;
    if (!ctx || !tree || !bytes) return MIRROR_ERR_ARG;
    if (tree->batch <= 0 || tree->n_nodes <= 0 || tree->n_nodes > MIRROR_MAX_NODES) return MIRROR_ERR_SHAPE;
    MirrorWsLayout L;
    mirror_ws_layout(ctx, (size_t)tree->batch * tree->n_nodes, &L, (size_t)tree->batch);
    size_t need = L.end_attn;
    if (what & (MIRROR_WS_LMHEAD | 4u)) need = L.end_lmhead;
    if (what & 32u) {
        // room for the candidate lists; and for the logits where the largest kappa could not be selected in the epilogue
        if (L.lm_topk_bytes && L.end_topk > need) need = L.end_topk;
        if (!mirror_lmhead_topk_fusable(ctx, (int)((size_t)tree->batch * tree->n_nodes), MIRROR_MAX_TOPK) && L.end_logits > need) need = L.end_logits;
    }
    if (what & 8u) need = L.end_logits > need ? L.end_logits : need;
    if (what & 16u) need = L.end_accept;
    *bytes = need;
    return MIRROR_OK;
}

extern "C" mirror_status mirror_set_workspace(mirror_ctx* ctx, void* dev_ptr, size_t bytes) {
    if (!ctx) return MIRROR_ERR_ARG;
    if (dev_ptr && ((uintptr_t)dev_ptr & 255)) return MIRROR_ERR_ARG;
    ctx->ws = dev_ptr;
    ctx->ws_bytes = dev_ptr ? bytes : 0;
    if (dev_ptr) {
        MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
        MIRROR_CUDA_OK(cudaMemset(dev_ptr, 0, bytes < kWsZeroedBytes ? bytes : kWsZeroedBytes));
    }
    return MIRROR_OK;
}

// ---------------------------------------------------------------------------------------------
// tensor maps
// ---------------------------------------------------------------------------------------------
mirror_status mirror_make_tmap(const mirror_ctx* ctx, CUtensorMap* map, const void* base, int rank,
                               const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box) {
    if (!ctx || !ctx->encode || !map || !base || rank < 1 || rank > 5) return MIRROR_ERR_ARG;
    if ((uintptr_t)base & 15) return MIRROR_ERR_ARG;
    cuuint64_t gdim[5];
    cuuint64_t gstride[4];
    cuuint32_t bdim[5], estride[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bdim[i] = box[i];
        estride[i] = 1;
        if (i + 1 < rank) {
            gstride[i] = strides_bytes[i];
            if (gstride[i] & 15) return MIRROR_ERR_SHAPE;
        }
    }
    CUresult r = ctx->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstride,
                             bdim, estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MIRROR_OK : MIRROR_ERR_CUDA;
}
