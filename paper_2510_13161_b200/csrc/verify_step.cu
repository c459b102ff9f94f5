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

extern "C" mirror_status mirror_attn_verify_fp8(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* q,
                                                const void* k_new_fp8, const void* v_new_fp8, const float* k_scale,
                                                const float* v_scale, float q_scale, void* out, float* lse_out, void* stream) {
    if (!ctx || !kv || !tree || !q || !k_new_fp8 || !v_new_fp8 || !k_scale || !v_scale || !out || !(q_scale > 0.f)) return MIRROR_ERR_ARG;
    if (ctx->desc.head_dim != 128) return MIRROR_ERR_UNSUPPORTED;
    mirror_status st = check_kv(ctx, kv, tree);
    if (st != MIRROR_OK) return st;
    if (((uintptr_t)q & 15) || ((uintptr_t)k_new_fp8 & 15) || ((uintptr_t)v_new_fp8 & 15) || ((uintptr_t)out & 15)) return MIRROR_ERR_ARG;
    MirrorTreeInfo ti;
    st = mirror_build_tree(tree, &ti);
    if (st != MIRROR_OK) return st;
    MirrorWsLayout L;
    mirror_ws_layout(ctx, (size_t)tree->batch * tree->n_nodes, &L);
    if (!ctx->ws || ctx->ws_bytes < L.end_attn) return MIRROR_ERR_WORKSPACE;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    uint8_t* ws = (uint8_t*)ctx->ws;
    const MirrorAttnFp8 f8 = {k_scale, v_scale, q_scale};
    return mirror_attn_launch(ctx, kv, tree, ti, q, k_new_fp8, v_new_fp8, out, lse_out, (float*)(ws + L.attn_partial),
                              (cudaStream_t)stream, &f8);
}

namespace {

struct HostIO {                       // host-buffer variant: pinned host inputs / outputs of one step
    const void* h_q;
    const void* h_k_new;
    const void* h_v_new;
    const int32_t* h_tokens;
    const mirror_accept_host_out* h_out;
};

constexpr int kHostChunks = kMirrorHostChunks;

mirror_status ensure_copy_stream(mirror_ctx* ctx) {
    if (ctx->copy_stream) return MIRROR_OK;
    MIRROR_CUDA_OK(cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
    for (int i = 0; i < kHostChunks + 1; ++i) MIRROR_CUDA_OK(cudaEventCreateWithFlags(&ctx->copy_ev[i], cudaEventDisableTiming));
    return MIRROR_OK;
}

mirror_status verify_step_impl(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* q, const void* k_new,
                               const void* v_new, const void* hidden, const void* W, const mirror_accept_in* acc,
                               const mirror_accept_out* out, void* attn_out, int32_t* argmax_out, void* stream, const HostIO* io,
                               const MirrorAttnFp8* f8 = nullptr) {
    if (f8 && io) return MIRROR_ERR_UNSUPPORTED;          // (the host-buffer step takes the bf16 cache)
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

    // (host-buffer variant) pieces of layers, copied on the second stream and attended to in that order
    int n_pieces = 0, piece_l0[kHostChunks] = {}, piece_l1[kHostChunks] = {};
    const size_t q_layer = M * (size_t)ctx->desc.n_q_heads * ctx->desc.head_dim * 2;        // bytes per layer
    const size_t kv_layer = M * (size_t)ctx->desc.n_kv_heads * ctx->desc.head_dim * 2;
    auto attend_piece = [&](int c) -> mirror_status {
        MIRROR_CUDA_OK(cudaStreamWaitEvent(s, ctx->copy_ev[c], 0));
        const int l0 = piece_l0[c], l1 = piece_l1[c];
        mirror_kv kv_c = *kv;
        kv_c.k_pool = (const __nv_bfloat16*)kv->k_pool + (size_t)l0 * kv->layer_stride;
        kv_c.v_pool = (const __nv_bfloat16*)kv->v_pool + (size_t)l0 * kv->layer_stride;
        kv_c.num_layers = l1 - l0;
        return mirror_attn_launch(ctx, &kv_c, tree, ti, (const uint8_t*)q + l0 * q_layer, (const uint8_t*)k_new + l0 * kv_layer,
                                  (const uint8_t*)v_new + l0 * kv_layer, (uint8_t*)attn_out + l0 * q_layer, nullptr,
                                  (float*)(ws + L.attn_partial), s);
    };
    const bool ev = ctx->stage_ev_on && !io;
    if (ev) MIRROR_CUDA_OK(cudaEventRecord(ctx->stage_ev[0], s));
    if (!io) {
        st = mirror_attn_launch(ctx, kv, tree, ti, q, k_new, v_new, attn_out, nullptr, (float*)(ws + L.attn_partial), s, f8);
        if (st != MIRROR_OK) return st;
    } else {
        // Host inputs.  The layers' attention problems are independent of one another and the LM head reads only the
        // last layer's output, so the last layer is copied and attended to first, the LM head and the acceptance follow
        // at once, and the other layers are copied in pieces on a second stream while the LM head streams its weights;
        // each piece is attended to as soon as it has landed (after the decision has gone back to the host).  The
        // copies start only after everything already queued on `stream` (the previous step may still read the staging
        // buffers).
        st = ensure_copy_stream(ctx);
        if (st != MIRROR_OK) return st;
        cudaStream_t cs = ctx->copy_stream;
        MIRROR_CUDA_OK(cudaEventRecord(ctx->copy_ev[kHostChunks], s));
        MIRROR_CUDA_OK(cudaStreamWaitEvent(cs, ctx->copy_ev[kHostChunks], 0));
        MIRROR_CUDA_OK(cudaMemcpyAsync((void*)tree->tokens, io->h_tokens, M * sizeof(int32_t), cudaMemcpyHostToDevice, cs));
        const int Lyr = kv->num_layers;
        n_pieces = 1 + (Lyr - 1 < kHostChunks - 1 ? Lyr - 1 : kHostChunks - 1);
        for (int c = 0; c < n_pieces; ++c) {
            // piece 0: the last layer; pieces 1..: the layers before it, in order
            const int l0 = c == 0 ? Lyr - 1 : (int)((long long)(Lyr - 1) * (c - 1) / (n_pieces - 1));
            const int l1 = c == 0 ? Lyr : (int)((long long)(Lyr - 1) * c / (n_pieces - 1));
            piece_l0[c] = l0; piece_l1[c] = l1;
            const size_t nl = (size_t)(l1 - l0);
            MIRROR_CUDA_OK(cudaMemcpyAsync((uint8_t*)q + l0 * q_layer, (const uint8_t*)io->h_q + l0 * q_layer, nl * q_layer,
                                           cudaMemcpyHostToDevice, cs));
            MIRROR_CUDA_OK(cudaMemcpyAsync((uint8_t*)k_new + l0 * kv_layer, (const uint8_t*)io->h_k_new + l0 * kv_layer, nl * kv_layer,
                                           cudaMemcpyHostToDevice, cs));
            MIRROR_CUDA_OK(cudaMemcpyAsync((uint8_t*)v_new + l0 * kv_layer, (const uint8_t*)io->h_v_new + l0 * kv_layer, nl * kv_layer,
                                           cudaMemcpyHostToDevice, cs));
            MIRROR_CUDA_OK(cudaEventRecord(ctx->copy_ev[c], cs));
        }
        st = attend_piece(0);
        if (st != MIRROR_OK) return st;
    }
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
    if (io && io->h_out) {
        const mirror_accept_host_out* h = io->h_out;
        const size_t B = (size_t)tree->batch;
        if (h->n_accepted) MIRROR_CUDA_OK(cudaMemcpyAsync(h->n_accepted, out->n_accepted, B * 4, cudaMemcpyDeviceToHost, s));
        if (h->best_branch) MIRROR_CUDA_OK(cudaMemcpyAsync(h->best_branch, out->best_branch, B * 4, cudaMemcpyDeviceToHost, s));
        if (h->n_emitted) MIRROR_CUDA_OK(cudaMemcpyAsync(h->n_emitted, out->n_emitted, B * 4, cudaMemcpyDeviceToHost, s));
        if (h->emitted) MIRROR_CUDA_OK(cudaMemcpyAsync(h->emitted, out->emitted, B * (size_t)(tree->gamma + 1) * 4, cudaMemcpyDeviceToHost, s));
    }
    for (int c = 1; c < n_pieces; ++c) {
        st = attend_piece(c);
        if (st != MIRROR_OK) return st;
    }
    return MIRROR_OK;
}

}  // namespace

extern "C" mirror_status mirror_verify_step(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree,
                                            const void* q, const void* k_new, const void* v_new, const void* hidden,
                                            const void* W, const mirror_accept_in* acc, const mirror_accept_out* out,
                                            void* attn_out, int32_t* argmax_out, void* stream) {
    return verify_step_impl(ctx, kv, tree, q, k_new, v_new, hidden, W, acc, out, attn_out, argmax_out, stream, nullptr);
}

extern "C" mirror_status mirror_verify_step_fp8(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* q,
                                                const void* k_new_fp8, const void* v_new_fp8, const float* k_scale,
                                                const float* v_scale, float q_scale, const void* hidden, const void* W,
                                                const mirror_accept_in* acc, const mirror_accept_out* out, void* attn_out,
                                                int32_t* argmax_out, void* stream) {
    if (!k_scale || !v_scale || !(q_scale > 0.f)) return MIRROR_ERR_ARG;
    if (ctx && ctx->desc.head_dim != 128) return MIRROR_ERR_UNSUPPORTED;
    const MirrorAttnFp8 f8 = {k_scale, v_scale, q_scale};
    return verify_step_impl(ctx, kv, tree, q, k_new_fp8, v_new_fp8, hidden, W, acc, out, attn_out, argmax_out, stream, nullptr, &f8);
}

extern "C" mirror_status mirror_verify_step_host(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* h_q,
                                                 const void* h_k_new, const void* h_v_new, const int32_t* h_tokens, void* d_q,
                                                 void* d_k_new, void* d_v_new, const void* hidden, const void* W,
                                                 const mirror_accept_in* acc, const mirror_accept_out* out,
                                                 const mirror_accept_host_out* h_out, void* attn_out, void* stream) {
    if (!h_q || !h_k_new || !h_v_new || !h_tokens) return MIRROR_ERR_ARG;
    HostIO io{h_q, h_k_new, h_v_new, h_tokens, h_out};
    return verify_step_impl(ctx, kv, tree, d_q, d_k_new, d_v_new, hidden, W, acc, out, attn_out, nullptr, stream, &io);
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
