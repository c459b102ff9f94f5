// Early-exit tap and its diagnostic (Sec. 3.1, Eq. 5 - Eq. 7): the LM head on intermediate hidden states, reduced to
// the Top-kappa message that the token channel carries (ids + bf16 log-probabilities), and the overlap mass of that
// message under the final distribution, whose complement is the probability of a fallback after a rejection at the
// window's first position (Proposition 1).
#include "mirror_internal.h"

namespace {

// One warp per row: Omega[row] = sum_k exp(logits[row][ids[row][k]] / T - lse[row]), lanes over k, fixed-order tree sum.
__global__ void overlap_mass_kernel(int M, int V, int kappa, float inv_T, const float* logits, const float* lse,
                                    const int32_t* ids, float* omega, int* status) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= M) return;
    float s = 0.f;
    for (int k = lane; k < kappa; k += 32) {
        const int id = ids[(size_t)row * kappa + k];
        if (id < 0 || id >= V) {
            if (atomicCAS(status, 0, MIRROR_DEV_CHECK) == 0) atomicExch(status + 1, 700 + k);
            continue;
        }
        s += expf(logits[(size_t)row * V + id] * inv_T - lse[row]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) omega[row] = s;
}

}  // namespace

extern "C" mirror_status mirror_early_exit_tap(mirror_ctx* ctx, const void* hidden_le, int M, const void* W, int kappa,
                                               int32_t* msg_ids, void* msg_logprob_bf16, void* stream) {
    if (!ctx || !hidden_le || !W || !msg_ids || !msg_logprob_bf16 || M <= 0 || kappa <= 0) return MIRROR_ERR_ARG;
    if (kappa > MIRROR_MAX_TOPK || kappa > ctx->desc.vocab) return MIRROR_ERR_SHAPE;
    if (((uintptr_t)hidden_le & 15) || ((uintptr_t)W & 15) || ((uintptr_t)msg_logprob_bf16 & 1)) return MIRROR_ERR_ARG;
    if (!ctx->ws) return MIRROR_ERR_WORKSPACE;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    MirrorWsLayout L;
    mirror_ws_layout(ctx, (size_t)M, &L);
    uint8_t* ws = (uint8_t*)ctx->ws;
    if (L.lm_topk_bytes && ctx->ws_bytes >= L.end_topk && mirror_lmhead_topk_fusable(ctx, M, kappa)) {
        // the Top-kappa is selected inside the GEMM's epilogue: the proxy's logits never reach memory
        return mirror_lmhead_launch(ctx, hidden_le, M, W, kappa, nullptr, nullptr, 0, nullptr, nullptr, nullptr, msg_ids, nullptr,
                                    nullptr, nullptr, ws + L.lm_partial, L.lm_partial_bytes, (float*)(ws + L.lse),
                                    (cudaStream_t)stream, nullptr, msg_logprob_bf16, ws + L.lm_topk, L.lm_topk_bytes);
    }
    if (ctx->ws_bytes < L.end_logits) return MIRROR_ERR_WORKSPACE;
    // a workspace without room for the candidate lists but with room for the logits: the selection runs over spilled logits
    return mirror_lmhead_launch(ctx, hidden_le, M, W, kappa, nullptr, nullptr, 0, nullptr, nullptr, nullptr, msg_ids, nullptr,
                                nullptr, (float*)(ws + L.logits), ws + L.lm_partial, L.lm_partial_bytes, (float*)(ws + L.lse),
                                (cudaStream_t)stream, nullptr, msg_logprob_bf16);
}

extern "C" mirror_status mirror_overlap_mass(mirror_ctx* ctx, const float* logits_final, const float* lse_final,
                                             const int32_t* msg_ids, int M, int kappa, float* omega, void* stream) {
    if (!ctx || !logits_final || !lse_final || !msg_ids || !omega || M <= 0 || kappa <= 0) return MIRROR_ERR_ARG;
    if (kappa > MIRROR_MAX_TOPK) return MIRROR_ERR_SHAPE;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    const int warps = 8;
    MIRROR_CUDA_OK(mirror_launch_pdl(overlap_mass_kernel, dim3((M + warps - 1) / warps), dim3(warps * 32), 0, (cudaStream_t)stream, M,
                                     ctx->desc.vocab, kappa, 1.0f / ctx->temperature, logits_final, lse_final, msg_ids, omega,
                                     ctx->d_status));
    ctx->launches += 1;
    MIRROR_CUDA_OK(cudaGetLastError());
    return MIRROR_OK;
}
