// The target's layers around the verify attention (the target forward of Sec. 3.1; the targets of Sec. 4.1 are
// pre-norm decoder stacks): per layer  RMSNorm -> Q/K/V projection -> rotary embedding -> branch-tree attention ->
// output projection + residual -> RMSNorm -> SiLU(gate) * up -> down projection + residual.
//
// The four projections run on the CTA-pair GEMM (lmhead_pair.cu, plain mode): with a few rows they are weight
// streams, and a projection with fewer 256-row output tiles than the GPU has CTA pairs is split along K so that every
// pair streams its share.  The GEMM leaves fp32 partial sums [slices][M][N]; a small "finish" kernel per projection
// adds the slices in a fixed order and applies what follows the projection in the layer, so no activation makes an
// extra trip through HBM: rotary embedding and the split into Q / K / V, residual add + the next RMSNorm, or the
// SiLU gate.  Activations are stored in bf16 (one rounding per stored tensor), sums are fp32.
// Every kernel is launched with programmatic stream serialization and waits for the kernel ahead before it touches
// global memory.
#include <math.h>

#include "mirror_internal.h"

namespace {

constexpr int kFinThreads = 256;

struct TreeDepths {
    int depth[MIRROR_MAX_NODES];
};

__device__ __forceinline__ float sum_slices(const float* partial, int slices, size_t slice_elems, size_t idx) {
    float a = 0.f;
    for (int s = 0; s < slices; ++s) a += partial[(size_t)s * slice_elems + idx];      // fixed order
    return a;
}

// cos / sin of every (row, frequency): row (b, i) sits at position prefix_len[b] + depth[i]; pair f turns by
// position * theta^(-2f/d).  Computed once per step in double precision (positions reach 10^5, where the fp32 product
// alone would be off by milliradians) and shared by all layers.
__global__ void rope_table_kernel(const int32_t* prefix_len, const TreeDepths td, int B, int n, int half, double theta,
                                  float2* cs) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= B * n * half) return;
    const int f = idx % half, row = idx / half;
    const int b = row / n, i = row % n;
    const double pos = (double)prefix_len[b] + (double)td.depth[i];
    const double inv_freq = exp(-(double)f / (double)half * log(theta));       // theta^(-2f/d), d = 2 * half
    double s, c;
    sincos(pos * inv_freq, &s, &c);
    cs[idx] = make_float2((float)c, (float)s);
}

// Q/K/V projection finish: split-K sum, rotary embedding on the query and key heads, bf16 stores into the step's
// [M, Hq, d] / [M, Hkv, d] tensors.  One block per (row, head), one thread per rotation pair (f, f + d/2); all
// slices of a thread's two columns are loaded before they are added (the loads are independent, the order of the sum
// is fixed).
__global__ void finish_qkv_kernel(const float* partial, int slices, int M, int Hq, int Hkv, int d, const float2* cs,
                                  __nv_bfloat16* q_out, __nv_bfloat16* k_out, __nv_bfloat16* v_out) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const int row = blockIdx.x, head = blockIdx.y, half = d >> 1, f = threadIdx.x;
    if (f >= half) return;
    const int N = (Hq + 2 * Hkv) * d;
    const size_t MN = (size_t)M * N;
    const float* p0 = partial + (size_t)row * N + (size_t)head * d + f;
    float a = 0.f, b = 0.f;
#pragma unroll 8
    for (int s = 0; s < slices; ++s) {
        a += p0[(size_t)s * MN];
        b += p0[(size_t)s * MN + half];
    }
    if (head < Hq + Hkv) {
        const float2 t = cs[(size_t)row * half + f];
        const float ra = a * t.x - b * t.y, rb = b * t.x + a * t.y;
        __nv_bfloat16* dst = head < Hq ? q_out + ((size_t)row * Hq + head) * d : k_out + ((size_t)row * Hkv + (head - Hq)) * d;
        dst[f] = __float2bfloat16_rn(ra);
        dst[f + half] = __float2bfloat16_rn(rb);
    } else {
        __nv_bfloat16* dst = v_out + ((size_t)row * Hkv + (head - Hq - Hkv)) * d;
        dst[f] = __float2bfloat16_rn(a);
        dst[f + half] = __float2bfloat16_rn(b);
    }
}

// Residual add + RMSNorm: r = residual + split-K sum, x_out = bf16(r); normed = bf16(x_out / sqrt(mean(x_out^2) + eps)
// * gamma) (from the ROUNDED x_out: what a later reader of x_out would compute).  One block of 1024 threads per row;
// a thread keeps its columns (every 1024th) in registers between the two passes and issues the loads of all slices
// of all its columns before adding them (in slice order).  partial == nullptr: plain RMSNorm of `residual`;
// gamma == nullptr: no norm.
constexpr int kNormThreads = 1024;
constexpr int kNormMaxCols = 16;              // columns per thread: rows of up to 16384 elements
template <int kNormCols, int kUnroll>         // kNormCols * 1024 >= H; kUnroll slices' loads in flight at a time
__global__ void __launch_bounds__(kNormThreads)
finish_residual_norm_kernel(const float* partial, int slices, int M, int H, const __nv_bfloat16* residual,
                            const __nv_bfloat16* gamma, float eps, __nv_bfloat16* x_out, __nv_bfloat16* normed) {
    __shared__ float s_red[kNormThreads / 32];
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const int row = blockIdx.x;
    const size_t MN = (size_t)M * H, base = (size_t)row * H;
    float r[kNormCols];
#pragma unroll
    for (int c = 0; c < kNormCols; ++c) {
        const int col = threadIdx.x + c * kNormThreads;
        r[c] = col < H ? __bfloat162float(residual[base + col]) : 0.f;
    }
    if (partial) {
        // several slices' loads in flight at a time; the additions stay in slice order
        for (int s0 = 0; s0 < slices; s0 += kUnroll) {
            float v[kUnroll][kNormCols];
#pragma unroll
            for (int k = 0; k < kUnroll; ++k)
#pragma unroll
                for (int c = 0; c < kNormCols; ++c) {
                    const int col = threadIdx.x + c * kNormThreads;
                    v[k][c] = (col < H && s0 + k < slices) ? partial[(size_t)(s0 + k) * MN + base + col] : 0.f;
                }
#pragma unroll
            for (int k = 0; k < kUnroll; ++k)
#pragma unroll
                for (int c = 0; c < kNormCols; ++c) r[c] += v[k][c];
        }
    }
    float ss = 0.f;
#pragma unroll
    for (int c = 0; c < kNormCols; ++c) {
        const int col = threadIdx.x + c * kNormThreads;
        if (col < H) {
            const __nv_bfloat16 xb = __float2bfloat16_rn(r[c]);
            if (x_out) x_out[base + col] = xb;
            r[c] = __bfloat162float(xb);
            ss = fmaf(r[c], r[c], ss);
        }
    }
    if (!gamma || !normed) return;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kNormThreads / 32; ++w) tot += s_red[w];               // same order in every thread
    const float rinv = 1.0f / sqrtf(tot / (float)H + eps);
#pragma unroll
    for (int c = 0; c < kNormCols; ++c) {
        const int col = threadIdx.x + c * kNormThreads;
        if (col < H) normed[base + col] = __float2bfloat16_rn(r[c] * rinv * __bfloat162float(gamma[col]));
    }
}

// Gated MLP finish: act[row, j] = bf16(silu(gate) * up), gate = sum of column j, up = sum of column I + j.
__global__ void __launch_bounds__(kFinThreads)
finish_swiglu_kernel(const float* partial, int slices, int M, int I, __nv_bfloat16* act) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const size_t MN = (size_t)M * 2 * I, total = (size_t)M * I;
    for (size_t idx = (size_t)blockIdx.x * kFinThreads + threadIdx.x; idx < total; idx += (size_t)gridDim.x * kFinThreads) {
        const size_t row = idx / I, j = idx - row * I;
        const float g = sum_slices(partial, slices, MN, row * 2 * I + j), u = sum_slices(partial, slices, MN, row * 2 * I + I + j);
        act[idx] = __float2bfloat16_rn(g / (1.0f + expf(-g)) * u);
    }
}

// Plain finish: out = bf16(split-K sum (+ residual)).
__global__ void __launch_bounds__(kFinThreads)
finish_store_kernel(const float* partial, int slices, size_t MN, const __nv_bfloat16* residual, __nv_bfloat16* out) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    for (size_t idx = (size_t)blockIdx.x * kFinThreads + threadIdx.x; idx < MN; idx += (size_t)gridDim.x * kFinThreads) {
        float r = sum_slices(partial, slices, MN, idx);
        if (residual) r += __bfloat162float(residual[idx]);
        out[idx] = __float2bfloat16_rn(r);
    }
}

cudaError_t launch_residual_norm(cudaStream_t s, const float* partial, int slices, int M, int H, const __nv_bfloat16* residual,
                                 const __nv_bfloat16* gamma, float eps, __nv_bfloat16* x_out, __nv_bfloat16* normed) {
    if (H <= 4 * kNormThreads)
        return mirror_launch_pdl(finish_residual_norm_kernel<4, 6>, dim3(M), dim3(kNormThreads), 0, s, partial, slices, M, H, residual, gamma,
                                 eps, x_out, normed);
    if (H <= 8 * kNormThreads)
        return mirror_launch_pdl(finish_residual_norm_kernel<8, 4>, dim3(M), dim3(kNormThreads), 0, s, partial, slices, M, H, residual, gamma,
                                 eps, x_out, normed);
    return mirror_launch_pdl(finish_residual_norm_kernel<16, 2>, dim3(M), dim3(kNormThreads), 0, s, partial, slices, M, H, residual, gamma,
                             eps, x_out, normed);
}

// Rows of the embedding table for the step's tokens: out[r] = table[tokens[r]] (16-byte copies; a token outside the
// vocabulary is reported and its row zeroed).
__global__ void embed_rows_kernel(const uint4* table, const int32_t* tokens, int M, int V, int row_vec, uint4* out, int* status) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const int r = blockIdx.x;
    const int t = tokens[r];
    const bool ok = t >= 0 && t < V;
    if (!ok && threadIdx.x == 0 && atomicCAS(status, 0, MIRROR_DEV_CHECK) == 0) atomicExch(status + 1, 900);
    for (int i = threadIdx.x; i < row_vec; i += blockDim.x)
        out[(size_t)r * row_vec + i] = ok ? table[(size_t)t * row_vec + i] : make_uint4(0, 0, 0, 0);
}

size_t partial_bytes_for(const mirror_ctx* ctx, int M, int N, int K) {
    return (size_t)mirror_linear_slices(ctx, M, N, K) * M * N * sizeof(float);
}

int grid_for(size_t elems, int num_sms) {
    size_t g = (elems + kFinThreads - 1) / kFinThreads;
    const size_t cap = (size_t)num_sms * 8;
    return (int)(g < cap ? (g > 0 ? g : 1) : cap);
}

struct TargetScratch {
    size_t partial = 0, partial_bytes = 0, cs = 0, h = 0, act = 0, xa = 0, xb = 0, total = 0;
};

TargetScratch target_scratch(const mirror_ctx* ctx, int M, int I) {
    const int H = ctx->desc.hidden, Hq = ctx->desc.n_q_heads, Hkv = ctx->desc.n_kv_heads, d = ctx->desc.head_dim;
    TargetScratch s;
    size_t pb = partial_bytes_for(ctx, M, (Hq + 2 * Hkv) * d, H);
    size_t x = partial_bytes_for(ctx, M, H, Hq * d);
    if (x > pb) pb = x;
    x = partial_bytes_for(ctx, M, 2 * I, H);
    if (x > pb) pb = x;
    x = partial_bytes_for(ctx, M, H, I);
    if (x > pb) pb = x;
    size_t at = 0;
    s.partial = at; s.partial_bytes = align_up(pb, 256); at += s.partial_bytes;
    s.cs = at; at += align_up((size_t)M * (d / 2) * sizeof(float2), 256);
    s.h = at; at += align_up((size_t)M * H * 2, 256);
    s.act = at; at += align_up((size_t)M * I * 2, 256);
    s.xa = at; at += align_up((size_t)M * H * 2, 256);
    s.xb = at; at += align_up((size_t)M * H * 2, 256);
    s.total = at;
    return s;
}

}  // namespace

extern "C" mirror_status mirror_linear_scratch_bytes(const mirror_ctx* ctx, int M, int N, int K, size_t* bytes) {
    if (!ctx || !bytes || M <= 0 || N <= 0 || K <= 0) return MIRROR_ERR_ARG;
    if (K % 64 != 0) return MIRROR_ERR_SHAPE;
    *bytes = partial_bytes_for(ctx, M, N, K);
    return MIRROR_OK;
}

extern "C" mirror_status mirror_linear(mirror_ctx* ctx, const void* x, int M, const void* W, int N, int K, const void* residual,
                                       void* out, void* scratch, size_t scratch_bytes, void* stream) {
    if (!ctx || !x || !W || !out || !scratch || M <= 0 || N <= 0 || K <= 0) return MIRROR_ERR_ARG;
    if (K % 64 != 0) return MIRROR_ERR_SHAPE;
    if (((uintptr_t)x & 15) || ((uintptr_t)W & 15) || ((uintptr_t)scratch & 15)) return MIRROR_ERR_ARG;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    cudaStream_t s = (cudaStream_t)stream;
    int slices = 0;
    mirror_status st = mirror_linear_partial_launch(ctx, x, M, W, N, K, (float*)scratch, scratch_bytes, s, &slices);
    if (st != MIRROR_OK) return st;
    const size_t MN = (size_t)M * N;
    MIRROR_CUDA_OK(mirror_launch_pdl(finish_store_kernel, dim3(grid_for(MN, ctx->num_sms)), dim3(kFinThreads), 0, s,
                                     (const float*)scratch, slices, MN, (const __nv_bfloat16*)residual, (__nv_bfloat16*)out));
    ctx->launches += 1;
    MIRROR_CUDA_OK(cudaGetLastError());
    return MIRROR_OK;
}

extern "C" mirror_status mirror_embed_rows(mirror_ctx* ctx, const void* table, const int32_t* tokens, int M, void* out, void* stream) {
    if (!ctx || !table || !tokens || !out || M <= 0) return MIRROR_ERR_ARG;
    const int H = ctx->desc.hidden, V = ctx->desc.vocab;
    if (H % 8 != 0) return MIRROR_ERR_SHAPE;
    if (((uintptr_t)table & 15) || ((uintptr_t)out & 15)) return MIRROR_ERR_ARG;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    MIRROR_CUDA_OK(mirror_launch_pdl(embed_rows_kernel, dim3(M), dim3(128), 0, (cudaStream_t)stream, (const uint4*)table, tokens, M, V, H / 8,
                                     (uint4*)out, ctx->d_status));
    ctx->launches += 1;
    MIRROR_CUDA_OK(cudaGetLastError());
    return MIRROR_OK;
}

extern "C" mirror_status mirror_rmsnorm(mirror_ctx* ctx, const void* x, const void* gamma, int M, int H, float eps, void* out,
                                        void* stream) {
    if (!ctx || !x || !gamma || !out || M <= 0 || H <= 0) return MIRROR_ERR_ARG;
    if (H > kNormThreads * kNormMaxCols) return MIRROR_ERR_SHAPE;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    MIRROR_CUDA_OK(launch_residual_norm((cudaStream_t)stream, nullptr, 0, M, H, (const __nv_bfloat16*)x, (const __nv_bfloat16*)gamma, eps,
                                        nullptr, (__nv_bfloat16*)out));
    ctx->launches += 1;
    MIRROR_CUDA_OK(cudaGetLastError());
    return MIRROR_OK;
}

extern "C" mirror_status mirror_target_scratch_bytes(const mirror_ctx* ctx, const mirror_tree* tree, const mirror_target* t,
                                                     size_t* bytes) {
    if (!ctx || !tree || !t || !bytes) return MIRROR_ERR_ARG;
    if (tree->batch <= 0 || tree->n_nodes <= 0 || tree->n_nodes > MIRROR_MAX_NODES || t->intermediate <= 0) return MIRROR_ERR_SHAPE;
    *bytes = target_scratch(ctx, tree->batch * tree->n_nodes, t->intermediate).total;
    return MIRROR_OK;
}

namespace {
// e4m3 cache: the cache's scales, one Q scale per layer (host), and where the codes of the new K/V rows go
struct TargetFp8 {
    const float* k_scale;      // device [L, Hkv]
    const float* v_scale;
    const float* q_scale;      // HOST [L]
    void* k_new8_out;          // device [L, B, n, Hkv, d] bytes
    void* v_new8_out;
};

mirror_status target_forward_impl(mirror_ctx* ctx, const mirror_target* t, const mirror_kv* kv, const mirror_tree* tree,
                                  const void* x, void* q_out, void* k_new_out, void* v_new_out, void* attn_out,
                                  void* x_out, void* hidden_out, void* scratch, size_t scratch_bytes, void* stream, const TargetFp8* f8) {
    if (!ctx || !t || !kv || !tree || !x || !q_out || !k_new_out || !v_new_out || !attn_out || !x_out || !hidden_out || !scratch)
        return MIRROR_ERR_ARG;
    if (!t->layers || !t->norm_final || t->n_layers <= 0 || t->n_layers > kv->num_layers) return MIRROR_ERR_ARG;
    const int H = ctx->desc.hidden, Hq = ctx->desc.n_q_heads, Hkv = ctx->desc.n_kv_heads, d = ctx->desc.head_dim, I = t->intermediate;
    if (I <= 0 || I % 64 != 0 || H % 64 != 0 || (Hq * d) % 64 != 0 || (d & 1)) return MIRROR_ERR_SHAPE;
    if (H > kNormThreads * kNormMaxCols || d / 2 > 1024) return MIRROR_ERR_SHAPE;
    if (!kv->k_pool || !kv->v_pool || !kv->page_table || !kv->prefix_len) return MIRROR_ERR_ARG;
    if (((uintptr_t)x & 15) || ((uintptr_t)scratch & 255)) return MIRROR_ERR_ARG;
    for (int l = 0; l < t->n_layers; ++l) {
        const mirror_layer_weights& w = t->layers[l];
        if (!w.w_qkv || !w.w_o || !w.w_gate_up || !w.w_down || !w.norm_attn || !w.norm_mlp) return MIRROR_ERR_ARG;
    }
    MirrorTreeInfo ti;
    mirror_status st = mirror_build_tree(tree, &ti);
    if (st != MIRROR_OK) return st;
    const int B = tree->batch, n = ti.n, M = B * n;
    const TargetScratch sc = target_scratch(ctx, M, I);
    if (scratch_bytes < sc.total) return MIRROR_ERR_WORKSPACE;
    MirrorWsLayout L;
    mirror_ws_layout(ctx, (size_t)M, &L);
    if (!ctx->ws || ctx->ws_bytes < L.end_attn) return MIRROR_ERR_WORKSPACE;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* base = (uint8_t*)scratch;
    float* partial = (float*)(base + sc.partial);
    float2* cs = (float2*)(base + sc.cs);
    __nv_bfloat16* h = (__nv_bfloat16*)(base + sc.h);
    __nv_bfloat16* act = (__nv_bfloat16*)(base + sc.act);
    __nv_bfloat16* xa = (__nv_bfloat16*)(base + sc.xa);
    __nv_bfloat16* xb = (__nv_bfloat16*)(base + sc.xb);

    TreeDepths td;
    for (int i = 0; i < MIRROR_MAX_NODES; ++i) td.depth[i] = i < n ? ti.depth[i] : 0;
    const int half = d / 2;
    MIRROR_CUDA_OK(mirror_launch_pdl(rope_table_kernel, dim3((M * half + 255) / 256), dim3(256), 0, s, kv->prefix_len, td, B, n, half,
                                     (double)t->rope_theta, cs));
    ctx->launches += 1;
    // the first layer's input norm; every later one comes out of the finish kernel of the layer before
    MIRROR_CUDA_OK(launch_residual_norm(s, nullptr, 0, M, H, (const __nv_bfloat16*)x, (const __nv_bfloat16*)t->layers[0].norm_attn, t->rms_eps,
                                        nullptr, h));
    ctx->launches += 1;

    const int Nqkv = (Hq + 2 * Hkv) * d;
    const size_t q_elems = (size_t)M * Hq * d, kv_elems = (size_t)M * Hkv * d;
    const __nv_bfloat16* x_cur = (const __nv_bfloat16*)x;
    for (int l = 0; l < t->n_layers; ++l) {
        const mirror_layer_weights& w = t->layers[l];
        const bool last = l + 1 == t->n_layers;
        __nv_bfloat16* q_l = (__nv_bfloat16*)q_out + (size_t)l * q_elems;
        __nv_bfloat16* k_l = (__nv_bfloat16*)k_new_out + (size_t)l * kv_elems;
        __nv_bfloat16* v_l = (__nv_bfloat16*)v_new_out + (size_t)l * kv_elems;
        __nv_bfloat16* a_l = (__nv_bfloat16*)attn_out + (size_t)l * q_elems;
        int slices = 0;
        // Q/K/V projection + rotary embedding
        st = mirror_linear_partial_launch(ctx, h, M, w.w_qkv, Nqkv, H, partial, sc.partial_bytes, s, &slices);
        if (st != MIRROR_OK) return st;
        MIRROR_CUDA_OK(mirror_launch_pdl(finish_qkv_kernel, dim3(M, Hq + 2 * Hkv), dim3(half), 0, s, (const float*)partial, slices, M, Hq, Hkv, d,
                                         (const float2*)cs, q_l, k_l, v_l));
        ctx->launches += 1;
        // attention of this layer over its slab of the cache
        mirror_kv kv_l = *kv;
        kv_l.num_layers = 1;
        if (!f8) {
            kv_l.k_pool = (const __nv_bfloat16*)kv->k_pool + (size_t)l * kv->layer_stride;
            kv_l.v_pool = (const __nv_bfloat16*)kv->v_pool + (size_t)l * kv->layer_stride;
            st = mirror_attn_launch(ctx, &kv_l, tree, ti, q_l, k_l, v_l, a_l, nullptr, (float*)((uint8_t*)ctx->ws + L.attn_partial), s);
        } else {
            // the layer's new K/V rows as codes under the cache's scales (the caller commits them), then the 8-bit attention
            uint8_t* k8_l = (uint8_t*)f8->k_new8_out + (size_t)l * kv_elems;
            uint8_t* v8_l = (uint8_t*)f8->v_new8_out + (size_t)l * kv_elems;
            st = mirror_kv_quantize_launch(ctx, k_l, 1, (int64_t)kv_elems, (int64_t)kv_elems, d, f8->k_scale + (size_t)l * Hkv, k8_l, s);
            if (st != MIRROR_OK) return st;
            st = mirror_kv_quantize_launch(ctx, v_l, 1, (int64_t)kv_elems, (int64_t)kv_elems, d, f8->v_scale + (size_t)l * Hkv, v8_l, s);
            if (st != MIRROR_OK) return st;
            kv_l.k_pool = (const uint8_t*)kv->k_pool + (size_t)l * kv->layer_stride;
            kv_l.v_pool = (const uint8_t*)kv->v_pool + (size_t)l * kv->layer_stride;
            const MirrorAttnFp8 a8 = {f8->k_scale + (size_t)l * Hkv, f8->v_scale + (size_t)l * Hkv, f8->q_scale[l]};
            st = mirror_attn_launch(ctx, &kv_l, tree, ti, q_l, k8_l, v8_l, a_l, nullptr, (float*)((uint8_t*)ctx->ws + L.attn_partial), s, &a8);
        }
        if (st != MIRROR_OK) return st;
        // output projection + residual + the MLP's norm
        st = mirror_linear_partial_launch(ctx, a_l, M, w.w_o, H, Hq * d, partial, sc.partial_bytes, s, &slices);
        if (st != MIRROR_OK) return st;
        MIRROR_CUDA_OK(launch_residual_norm(s, partial, slices, M, H, x_cur, (const __nv_bfloat16*)w.norm_mlp, t->rms_eps, xa, h));
        ctx->launches += 1;
        // gate / up projection + SiLU gate
        st = mirror_linear_partial_launch(ctx, h, M, w.w_gate_up, 2 * I, H, partial, sc.partial_bytes, s, &slices);
        if (st != MIRROR_OK) return st;
        MIRROR_CUDA_OK(mirror_launch_pdl(finish_swiglu_kernel, dim3(grid_for((size_t)M * I, ctx->num_sms)), dim3(kFinThreads), 0, s,
                                         (const float*)partial, slices, M, I, act));
        ctx->launches += 1;
        // down projection + residual + the next layer's (or the final) norm
        st = mirror_linear_partial_launch(ctx, act, M, w.w_down, H, I, partial, sc.partial_bytes, s, &slices);
        if (st != MIRROR_OK) return st;
        const void* g_next = last ? t->norm_final : t->layers[l + 1].norm_attn;
        __nv_bfloat16* x_new = last ? (__nv_bfloat16*)x_out : xb;
        MIRROR_CUDA_OK(launch_residual_norm(s, partial, slices, M, H, xa, (const __nv_bfloat16*)g_next, t->rms_eps, x_new,
                                            last ? (__nv_bfloat16*)hidden_out : h));
        ctx->launches += 1;
        x_cur = xb;
    }
    MIRROR_CUDA_OK(cudaGetLastError());
    return MIRROR_OK;
}

}  // namespace

extern "C" mirror_status mirror_target_forward(mirror_ctx* ctx, const mirror_target* t, const mirror_kv* kv, const mirror_tree* tree,
                                               const void* x, void* q_out, void* k_new_out, void* v_new_out, void* attn_out,
                                               void* x_out, void* hidden_out, void* scratch, size_t scratch_bytes, void* stream) {
    return target_forward_impl(ctx, t, kv, tree, x, q_out, k_new_out, v_new_out, attn_out, x_out, hidden_out, scratch, scratch_bytes,
                               stream, nullptr);
}

extern "C" mirror_status mirror_target_forward_fp8(mirror_ctx* ctx, const mirror_target* t, const mirror_kv* kv, const mirror_tree* tree,
                                                   const void* x, const float* k_scale, const float* v_scale, const float* h_q_scale,
                                                   void* q_out, void* k_new_out, void* v_new_out, void* k_new8_out, void* v_new8_out,
                                                   void* attn_out, void* x_out, void* hidden_out, void* scratch, size_t scratch_bytes,
                                                   void* stream) {
    if (!k_scale || !v_scale || !h_q_scale || !k_new8_out || !v_new8_out) return MIRROR_ERR_ARG;
    if (ctx && ctx->desc.head_dim != 128) return MIRROR_ERR_UNSUPPORTED;
    if (t) for (int l = 0; l < t->n_layers; ++l) if (!(h_q_scale[l] > 0.f)) return MIRROR_ERR_ARG;
    const TargetFp8 f8 = {k_scale, v_scale, h_q_scale, k_new8_out, v_new8_out};
    return target_forward_impl(ctx, t, kv, tree, x, q_out, k_new_out, v_new_out, attn_out, x_out, hidden_out, scratch, scratch_bytes,
                               stream, &f8);
}
