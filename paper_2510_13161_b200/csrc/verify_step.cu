// Public entry points for attention and for the fused verify step (attention over all layers ->
// LM head with fused reductions -> acceptance), all enqueued on one stream.
#include "mirror_internal.h"

namespace {

mirror_status check_kv(const mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree) {
    if (!kv->k_pool || !kv->v_pool || !kv->page_table || !kv->prefix_len) return MIRROR_ERR_ARG;
    if (kv->num_layers <= 0 || kv->num_pages <= 0 || kv->max_pages_per_req <= 0) return MIRROR_ERR_ARG;
    if (((uintptr_t)kv->k_pool & 15) || ((uintptr_t)kv->v_pool & 15)) return MIRROR_ERR_ARG;
    const int64_t page_elems = (int64_t)ctx->desc.n_kv_heads * ctx->desc.page_size * ctx->desc.head_dim;
    if (kv->num_layers > 1 && (kv->layer_stride < (int64_t)kv->num_pages * page_elems)) return MIRROR_ERR_SHAPE;
    if (kv->layer_stride % page_elems != 0) return MIRROR_ERR_UNSUPPORTED;
    (void)tree;
    return MIRROR_OK;
}

}  // namespace

extern "C" mirror_status mirror_attn_verify(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree,
                                            const void* q, const void* k_new, const void* v_new, void* out,
                                            float* lse_out, void* stream) {
    if (!ctx || !kv || !tree || !q || !k_new || !v_new || !out) return MIRROR_ERR_ARG;
    mirror_status st = check_kv(ctx, kv, tree);
    if (st != MIRROR_OK) return st;
    if (((uintptr_t)q & 15) || ((uintptr_t)k_new & 15) || ((uintptr_t)v_new & 15) || ((uintptr_t)out & 15)) return MIRROR_ERR_ARG;
    MirrorTreeInfo ti;
    st = mirror_build_tree(tree, &ti);
    if (st != MIRROR_OK) return st;
    MirrorWsLayout L;
    mirror_ws_layout(ctx, (size_t)tree->batch * tree->n_nodes, &L);
    if (!ctx->ws || ctx->ws_bytes < L.end_attn) return MIRROR_ERR_WORKSPACE;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    uint8_t* ws = (uint8_t*)ctx->ws;
    return mirror_attn_launch(ctx, kv, tree, ti, q, k_new, v_new, out, lse_out, (float*)(ws + L.attn_partial), (cudaStream_t)stream);
}

extern "C" mirror_status mirror_verify_step(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree,
                                            const void* q, const void* k_new, const void* v_new, const void* hidden,
                                            const void* W, const mirror_accept_in* acc, const mirror_accept_out* out,
                                            void* attn_out, int32_t* argmax_out, void* stream) {
    if (!ctx || !kv || !tree || !q || !k_new || !v_new || !W || !acc || !out || !attn_out || !tree->tokens) return MIRROR_ERR_ARG;
    if (!out->n_accepted || !out->best_branch || !out->n_emitted || !out->emitted || !out->accepted_nodes ||
        !out->decide_row || !out->reuse_slot)
        return MIRROR_ERR_ARG;
    mirror_status st = check_kv(ctx, kv, tree);
    if (st != MIRROR_OK) return st;
    const bool spec = acc->mode == MIRROR_ACCEPT_SPEC_SAMPLING || acc->mode == MIRROR_ACCEPT_SPEC_TREE;
    if (!spec && acc->mode != MIRROR_ACCEPT_GREEDY) return MIRROR_ERR_ARG;
    if (spec && (!acc->u_accept || !acc->u_resample || (tree->n_nodes > 1 && !acc->q_probs))) return MIRROR_ERR_ARG;
    if (!hidden && ctx->desc.n_q_heads * ctx->desc.head_dim != ctx->desc.hidden) return MIRROR_ERR_SHAPE;
    MirrorTreeInfo ti;
    st = mirror_build_tree(tree, &ti);
    if (st != MIRROR_OK) return st;
    const size_t M = (size_t)tree->batch * tree->n_nodes;
    MirrorWsLayout L;
    mirror_ws_layout(ctx, M, &L, (size_t)tree->batch);
    if (!ctx->ws || ctx->ws_bytes < (spec ? L.end_logits : L.end_lmhead)) return MIRROR_ERR_WORKSPACE;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    uint8_t* ws = (uint8_t*)ctx->ws;
    cudaStream_t s = (cudaStream_t)stream;

    const bool ev = ctx->stage_ev_on;
    if (ev) MIRROR_CUDA_OK(cudaEventRecord(ctx->stage_ev[0], s));
    st = mirror_attn_launch(ctx, kv, tree, ti, q, k_new, v_new, attn_out, nullptr, (float*)(ws + L.attn_partial), s);
    if (st != MIRROR_OK) return st;
    if (ev) MIRROR_CUDA_OK(cudaEventRecord(ctx->stage_ev[1], s));

    // LM-head rows: the given hidden states, else the last layer's attention output ([B*n, Hq*d] == [M, H])
    const void* rows = hidden;
    if (!rows) {
        const size_t layer_elems = M * (size_t)ctx->desc.n_q_heads * ctx->desc.head_dim;
        rows = (const __nv_bfloat16*)attn_out + (size_t)(kv->num_layers - 1) * layer_elems;
    }
    int32_t* d_argmax = argmax_out ? argmax_out : (int32_t*)(ws + L.argmax);
    float* d_lse = (float*)(ws + L.lse);
    float* d_logits = spec ? (float*)(ws + L.logits) : nullptr;
    st = mirror_lmhead_launch(ctx, rows, (int)M, W, 0, nullptr, nullptr, 0, d_argmax, nullptr, spec ? d_lse : nullptr, nullptr,
                              nullptr, nullptr, d_logits, ws + L.lm_partial, L.lm_partial_bytes, d_lse, s,
                              ev ? ctx->stage_ev[2] : nullptr);
    if (st != MIRROR_OK) return st;

    mirror_accept_in in = *acc;
    in.target_argmax = d_argmax;
    in.logits = d_logits;
    in.lse = d_lse;
    // the tree rule keeps its running distribution in the workspace when the caller sized it for that
    double* tree_scratch = (acc->mode == MIRROR_ACCEPT_SPEC_TREE && ctx->ws_bytes >= L.end_accept) ? (double*)(ws + L.accept_scratch) : nullptr;
    st = mirror_accept_launch(ctx, tree, ti, &in, out, s, tree_scratch);
    if (st != MIRROR_OK) return st;
    if (ev) MIRROR_CUDA_OK(cudaEventRecord(ctx->stage_ev[3], s));
    return MIRROR_OK;
}

extern "C" mirror_status mirror_set_stage_events(mirror_ctx* ctx, void* const* events4) {
    if (!ctx) return MIRROR_ERR_ARG;
    ctx->stage_ev_on = false;
    if (!events4) return MIRROR_OK;
    for (int i = 0; i < 4; ++i) {
        if (!events4[i]) return MIRROR_ERR_ARG;
        ctx->stage_ev[i] = (cudaEvent_t)events4[i];
    }
    ctx->stage_ev_on = true;
    return MIRROR_OK;
}
