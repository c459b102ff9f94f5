// Roll-forward of the paged KV cache after a verify step (Sec. 3.1: the target commits the accepted prefix of the
// window and rolls its state forward): the K/V rows of the root and of the accepted nodes of the chosen branch, in
// path order, become tokens prefix_len .. prefix_len + A of every layer and KV head, and the prefix grows by A + 1.
// Pure data movement: 2 * L * (A + 1) * Hkv * d bf16 values per request.
#include "mirror_internal.h"

namespace {

struct CommitParams {
    int L, B, n, Hkv, d, gamma, max_pages, num_pages;
    long long layer_stride;               // elements between the layers' pools
    __nv_bfloat16* k_pool;
    __nv_bfloat16* v_pool;
    const __nv_bfloat16* k_new;           // [L, B, n, Hkv, d]
    const __nv_bfloat16* v_new;
    const int32_t* page_table;
    const int32_t* prefix_len;
    const int32_t* accepted_nodes;        // [B, gamma]
    const int32_t* n_accepted;            // [B]
    int* status;
};

// grid (L, B): the block copies the (A + 1) x Hkv rows of d values of both tensors with 16-byte accesses
__global__ void __launch_bounds__(256) kv_commit_kernel(const CommitParams p) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const int layer = blockIdx.x, b = blockIdx.y;
    int A = p.n_accepted[b];
    if (A < 0 || A > p.gamma) { if (threadIdx.x == 0 && atomicCAS(p.status, 0, MIRROR_DEV_CHECK) == 0) atomicExch(p.status + 1, 800); A = 0; }
    const int len = p.prefix_len[b];
    const int chunks_per_row = p.d / 8;                       // 16-byte chunks of one (token, head) row
    const int total = (A + 1) * p.Hkv * chunks_per_row;
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
        const int cc = i % chunks_per_row, h = (i / chunks_per_row) % p.Hkv, j = i / (chunks_per_row * p.Hkv);
        const int node = (j == 0) ? 0 : p.accepted_nodes[(size_t)b * p.gamma + j - 1];
        const int pos = len + j;
        bool ok = len >= 0 && node >= 0 && node < p.n && pos < p.max_pages * 16;
        int page = ok ? p.page_table[(size_t)b * p.max_pages + pos / 16] : -1;
        ok = ok && page >= 0 && page < p.num_pages;
        if (!ok) {                                            // reported, not written
            if (atomicCAS(p.status, 0, MIRROR_DEV_CHECK) == 0) atomicExch(p.status + 1, 801);
            continue;
        }
        const size_t src = ((((size_t)layer * p.B + b) * p.n + node) * p.Hkv + h) * p.d + cc * 8;
        const size_t dst = (size_t)layer * p.layer_stride + (((size_t)page * p.Hkv + h) * 16 + pos % 16) * p.d + cc * 8;
        *reinterpret_cast<uint4*>(p.k_pool + dst) = *reinterpret_cast<const uint4*>(p.k_new + src);
        *reinterpret_cast<uint4*>(p.v_pool + dst) = *reinterpret_cast<const uint4*>(p.v_new + src);
    }
}

// after every layer has read the old lengths
__global__ void kv_advance_kernel(int B, int gamma, const int32_t* n_accepted, int32_t* prefix_len) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int A = n_accepted[b];
    prefix_len[b] += ((A < 0 || A > gamma) ? 0 : A) + 1;
}

}  // namespace

// elem_bytes 2: bf16 cache.  1: e4m3 codes; a row of d codes is moved as d / 2 16-bit units, the layout is the same.
static mirror_status kv_commit_impl(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* k_new,
                                    const void* v_new, const int32_t* accepted_nodes, const int32_t* n_accepted,
                                    int32_t* prefix_len, void* stream, int elem_bytes) {
    if (!ctx || !kv || !tree || !k_new || !v_new || !accepted_nodes || !n_accepted || !prefix_len) return MIRROR_ERR_ARG;
    if (!kv->k_pool || !kv->v_pool || !kv->page_table) return MIRROR_ERR_ARG;
    if (tree->batch <= 0 || tree->n_nodes <= 0 || tree->n_nodes > MIRROR_MAX_NODES || tree->gamma < 0 || tree->gamma > MIRROR_MAX_DEPTH)
        return MIRROR_ERR_SHAPE;
    if (kv->num_layers <= 0 || kv->num_pages <= 0 || kv->max_pages_per_req <= 0) return MIRROR_ERR_ARG;
    if (((uintptr_t)k_new & 15) || ((uintptr_t)v_new & 15) || ((uintptr_t)kv->k_pool & 15) || ((uintptr_t)kv->v_pool & 15)) return MIRROR_ERR_ARG;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    CommitParams p;
    p.L = kv->num_layers; p.B = tree->batch; p.n = tree->n_nodes; p.Hkv = ctx->desc.n_kv_heads;
    p.d = ctx->desc.head_dim * elem_bytes / 2;
    if (kv->layer_stride * elem_bytes % 2 != 0) return MIRROR_ERR_SHAPE;
    p.gamma = tree->gamma; p.max_pages = kv->max_pages_per_req; p.num_pages = kv->num_pages;
    p.layer_stride = kv->layer_stride * elem_bytes / 2;
    p.k_pool = (__nv_bfloat16*)const_cast<void*>(kv->k_pool);
    p.v_pool = (__nv_bfloat16*)const_cast<void*>(kv->v_pool);
    p.k_new = (const __nv_bfloat16*)k_new; p.v_new = (const __nv_bfloat16*)v_new;
    p.page_table = kv->page_table; p.prefix_len = prefix_len;
    p.accepted_nodes = accepted_nodes; p.n_accepted = n_accepted;
    p.status = ctx->d_status;
    cudaStream_t s = (cudaStream_t)stream;
    MIRROR_CUDA_OK(mirror_launch_pdl(kv_commit_kernel, dim3((unsigned)p.L, (unsigned)p.B), dim3(256), 0, s, p));
    MIRROR_CUDA_OK(mirror_launch_pdl(kv_advance_kernel, dim3((unsigned)((p.B + 127) / 128)), dim3(128), 0, s, p.B, p.gamma, n_accepted, prefix_len));
    ctx->launches += 2;
    MIRROR_CUDA_OK(cudaGetLastError());
    return MIRROR_OK;
}

extern "C" mirror_status mirror_kv_commit(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* k_new,
                                          const void* v_new, const int32_t* accepted_nodes, const int32_t* n_accepted,
                                          int32_t* prefix_len, void* stream) {
    return kv_commit_impl(ctx, kv, tree, k_new, v_new, accepted_nodes, n_accepted, prefix_len, stream, 2);
}

extern "C" mirror_status mirror_kv_commit_fp8(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* k_new_fp8,
                                              const void* v_new_fp8, const int32_t* accepted_nodes, const int32_t* n_accepted,
                                              int32_t* prefix_len, void* stream) {
    return kv_commit_impl(ctx, kv, tree, k_new_fp8, v_new_fp8, accepted_nodes, n_accepted, prefix_len, stream, 1);
}
