// e4m3 KV cache: scales per (layer, KV head) and the codes of a bf16 K or V tensor under them.
//
// The paper states no storage precision for the target's cache (Section 3, Eq. 1); the 8-bit cache is this library's own
// option.  A tensor is addressed as [layer][...][head][inner]: `inner` consecutive elements belong to one head (a page
// of one head in a pool: page_size * d; one token's row of the tree's own K/V: d), heads cycle fastest above that.
//   scale[layer, head] = max|x| / 448 over that layer's and head's elements (1 if all are zero), in fp32
//   code = e4m3(x / scale), fp32 division, round to nearest even, saturating at +-448
#include <cuda_fp8.h>

#include "mirror_internal.h"

namespace {

struct KvQuantParams {
    const __nv_bfloat16* x;
    uint8_t* out;
    float* scale;             // [L, Hkv]
    int L, Hkv;
    long long layer_stride;   // elements between layers (input and output alike)
    long long layer_elems;    // elements of a layer that are in use
    int inner;                // consecutive elements of one head (a multiple of 8)
};

// amax per (layer, head) into scale[] as the bit pattern of a non-negative float (ordered like an integer)
__global__ void __launch_bounds__(256) kv_amax_kernel(const KvQuantParams p) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const long long chunks_per_layer = p.layer_elems / 8;
    const long long total = chunks_per_layer * p.L;
    int key = -1;
    float amax = 0.f;
    for (long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x; c < total; c += (long long)gridDim.x * blockDim.x) {
        const int l = (int)(c / chunks_per_layer);
        const long long e = (c - (long long)l * chunks_per_layer) * 8;
        const int h = (int)((e / p.inner) % p.Hkv);
        const int k = l * p.Hkv + h;
        if (k != key) {
            if (key >= 0 && amax > 0.f) atomicMax((int*)p.scale + key, __float_as_int(amax));
            key = k;
            amax = 0.f;
        }
        const uint4 v = *reinterpret_cast<const uint4*>(p.x + (size_t)l * p.layer_stride + e);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            amax = fmaxf(amax, fabsf(__uint_as_float(w[i] << 16)));
            amax = fmaxf(amax, fabsf(__uint_as_float(w[i] & 0xffff0000u)));
        }
    }
    if (key >= 0 && amax > 0.f) atomicMax((int*)p.scale + key, __float_as_int(amax));
}

__global__ void kv_scale_finish_kernel(float* scale, int n) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        const float a = scale[i];
        scale[i] = a > 0.f ? __fdiv_rn(a, 448.f) : 1.f;
    }
}

__global__ void __launch_bounds__(256) kv_quantize_kernel(const KvQuantParams p) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const long long chunks_per_layer = p.layer_elems / 8;
    const long long total = chunks_per_layer * p.L;
    for (long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x; c < total; c += (long long)gridDim.x * blockDim.x) {
        const int l = (int)(c / chunks_per_layer);
        const long long e = (c - (long long)l * chunks_per_layer) * 8;
        const int h = (int)((e / p.inner) % p.Hkv);
        const float sc = __ldg(p.scale + l * p.Hkv + h);
        const uint4 v = *reinterpret_cast<const uint4*>(p.x + (size_t)l * p.layer_stride + e);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[2] = {0, 0};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t c0 = __nv_cvt_float_to_fp8(__fdiv_rn(__uint_as_float(w[i] << 16), sc), __NV_SATFINITE, __NV_E4M3);
            const uint32_t c1 = __nv_cvt_float_to_fp8(__fdiv_rn(__uint_as_float(w[i] & 0xffff0000u), sc), __NV_SATFINITE, __NV_E4M3);
            o[i >> 1] |= (c0 | (c1 << 8)) << ((i & 1) * 16);
        }
        *reinterpret_cast<uint2*>(p.out + (size_t)l * p.layer_stride + e) = make_uint2(o[0], o[1]);
    }
}

mirror_status fill(const mirror_ctx* ctx, KvQuantParams* p, const void* x, int n_layers, int64_t layer_stride, int64_t layer_elems,
                   int inner, float* scale) {
    if (!ctx || !x || !scale || n_layers <= 0 || layer_elems <= 0 || inner <= 0) return MIRROR_ERR_ARG;
    if (inner % 8 != 0 || layer_elems % ((int64_t)inner * ctx->desc.n_kv_heads) != 0) return MIRROR_ERR_SHAPE;
    if (n_layers > 1 && (layer_stride < layer_elems || layer_stride % 8 != 0)) return MIRROR_ERR_SHAPE;
    if ((uintptr_t)x & 15) return MIRROR_ERR_ARG;
    p->x = (const __nv_bfloat16*)x;
    p->out = nullptr;
    p->scale = scale;
    p->L = n_layers;
    p->Hkv = ctx->desc.n_kv_heads;
    p->layer_stride = layer_stride;
    p->layer_elems = layer_elems;
    p->inner = inner;
    return MIRROR_OK;
}

unsigned grid_for(const mirror_ctx* ctx, const KvQuantParams& p) {
    const long long chunks = p.layer_elems / 8 * p.L;
    const long long blocks = (chunks + 255) / 256;
    const long long cap = (long long)ctx->num_sms * 8;
    return (unsigned)(blocks < cap ? blocks : cap);
}

}  // namespace

extern "C" mirror_status mirror_kv_scales_fp8(mirror_ctx* ctx, const void* x, int n_layers, int64_t layer_stride,
                                              int64_t layer_elems, int inner, float* scale, void* stream) {
    KvQuantParams p;
    mirror_status st = fill(ctx, &p, x, n_layers, layer_stride, layer_elems, inner, scale);
    if (st != MIRROR_OK) return st;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    cudaStream_t s = (cudaStream_t)stream;
    const int n = n_layers * p.Hkv;
    MIRROR_CUDA_OK(cudaMemsetAsync(scale, 0, sizeof(float) * n, s));
    kv_amax_kernel<<<grid_for(ctx, p), 256, 0, s>>>(p);
    MIRROR_CUDA_OK(cudaGetLastError());
    kv_scale_finish_kernel<<<(n + 255) / 256, 256, 0, s>>>(scale, n);
    MIRROR_CUDA_OK(cudaGetLastError());
    ctx->launches += 2;
    return MIRROR_OK;
}

mirror_status mirror_kv_quantize_launch(mirror_ctx* ctx, const void* x, int n_layers, int64_t layer_stride, int64_t layer_elems,
                                       int inner, const float* scale, void* out_fp8, cudaStream_t stream) {
    KvQuantParams p;
    mirror_status st = fill(ctx, &p, x, n_layers, layer_stride, layer_elems, inner, const_cast<float*>(scale));
    if (st != MIRROR_OK) return st;
    if (!out_fp8 || ((uintptr_t)out_fp8 & 7)) return MIRROR_ERR_ARG;
    p.out = (uint8_t*)out_fp8;
    MIRROR_CUDA_OK(mirror_launch_pdl(kv_quantize_kernel, dim3(grid_for(ctx, p)), dim3(256), 0, stream, p));
    MIRROR_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return MIRROR_OK;
}

extern "C" mirror_status mirror_kv_quantize_fp8(mirror_ctx* ctx, const void* x, int n_layers, int64_t layer_stride,
                                                int64_t layer_elems, int inner, const float* scale, void* out_fp8, void* stream) {
    KvQuantParams p;
    mirror_status st = fill(ctx, &p, x, n_layers, layer_stride, layer_elems, inner, const_cast<float*>(scale));
    if (st != MIRROR_OK) return st;
    if (!out_fp8 || ((uintptr_t)out_fp8 & 7)) return MIRROR_ERR_ARG;
    p.out = (uint8_t*)out_fp8;
    MIRROR_CUDA_OK(cudaSetDevice(ctx->device));
    kv_quantize_kernel<<<grid_for(ctx, p), 256, 0, (cudaStream_t)stream>>>(p);
    MIRROR_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return MIRROR_OK;
}
