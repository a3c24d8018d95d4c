// CUDA-core rotary embedding + K/V append and causal attention for the rows of one step.
// The work done for a query at absolute position p is a function of p alone (positions are
// dealt to warps by p mod 4, partial softmax states are merged in warp order), so a row's
// result does not depend on which other rows share the step.
#include "kernels.h"

namespace llma {

// qkv[r] = [q (HD) | k (HD) | v (HD)] fp32.  Rotates q and k in place (pair (i, i+hd/2),
// angle pos * theta^(-2i/hd) from the host-built table) and stores k, v into the cache.
template <typename T>
__global__ void qkv_post_kernel(ModelDims dims, int layer, const RowDesc* __restrict__ rows, float* __restrict__ qkv,
                                const float* __restrict__ rope_cos, const float* __restrict__ rope_sin,
                                T* __restrict__ kcache, T* __restrict__ vcache) {
    pdl_trigger();
    pdl_wait();
    const int r = blockIdx.x, head = blockIdx.y;
    const int pos = rows->pos[r];
    if (pos < 0) return;
    const int hd = dims.head_dim, half = hd / 2, HD = dims.hd_total;
    const int seq = rows->seq[r];
    float* q = qkv + (int64_t)r * 3 * HD + head * hd;
    float* k = q + HD;
    const float* v = q + 2 * HD;
    const int64_t crow = kv_row_index(dims, layer, seq, head, pos) * hd;
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        const float c = rope_cos[(int64_t)pos * half + i], s = rope_sin[(int64_t)pos * half + i];
        const float qa = q[i], qb = q[i + half];
        q[i] = qa * c - qb * s;
        q[i + half] = qa * s + qb * c;
        const float ka = k[i], kb = k[i + half];
        kcache[crow + i] = from_f32<T>(ka * c - kb * s);
        kcache[crow + i + half] = from_f32<T>(ka * s + kb * c);
        vcache[crow + i] = from_f32<T>(v[i]);
        vcache[crow + i + half] = from_f32<T>(v[i + half]);
    }
}

template <typename T, int EPL>  // EPL = head_dim / 32 elements per lane
__global__ void __launch_bounds__(128) attention_simt_kernel(ModelDims dims, int layer,
                                                             const RowDesc* __restrict__ rows,
                                                             const float* __restrict__ qkv,
                                                             const T* __restrict__ kcache,
                                                             const T* __restrict__ vcache, void* __restrict__ attn_out,
                                                             int act_layout) {
    pdl_trigger();
    pdl_wait();
    const int head = blockIdx.x, r = blockIdx.y;
    const int pos = rows->pos[r];
    if (pos < 0) return;
    const int hd = dims.head_dim, HD = dims.hd_total;
    const int seq = rows->seq[r];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float scale = rsqrtf((float)hd);
    const float* q = qkv + (int64_t)r * 3 * HD + head * hd + lane * EPL;
    float qv[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) qv[e] = q[e];
    const int64_t base = kv_row_index(dims, layer, seq, head, 0) * hd;
    const T* K = kcache + base + lane * EPL;
    const T* V = vcache + base + lane * EPL;

    float m = -INFINITY, l = 0.f, acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    for (int p = warp; p <= pos; p += 4) {
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) s = fmaf(qv[e], to_f32<T>(K[(int64_t)p * hd + e]), s);
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        s *= scale;
        const float mn = fmaxf(m, s);
        const float corr = expf(m - mn), pe = expf(s - mn);
        l = l * corr + pe;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = acc[e] * corr + pe * to_f32<T>(V[(int64_t)p * hd + e]);
        m = mn;
    }
    __shared__ float sm[4], sl[4], sacc[4][128];
    if (lane == 0) { sm[warp] = m; sl[warp] = l; }
#pragma unroll
    for (int e = 0; e < EPL; ++e) sacc[warp][lane * EPL + e] = acc[e];
    __syncthreads();
    if (warp == 0) {
        float M = sm[0];
        for (int w = 1; w < 4; ++w) M = fmaxf(M, sm[w]);
        float den = 0.f, num[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) num[e] = 0.f;
        for (int w = 0; w < 4; ++w) {
            const float f = expf(sm[w] - M);  // 0 for a warp that saw no position
            den += f * sl[w];
#pragma unroll
            for (int e = 0; e < EPL; ++e) num[e] += f * sacc[w][lane * EPL + e];
        }
#pragma unroll
        for (int e = 0; e < EPL; ++e) store_act(attn_out, act_layout, dims.row_cap, r, head * hd + lane * EPL + e, HD, num[e] / den);
    }
}

void launch_qkv_post(cudaStream_t st, bool bf16, const ModelDims& dims, int layer, int n_rows, const RowDesc* rows,
                     float* qkv, const float* rope_cos, const float* rope_sin, void* kcache, void* vcache) {
    dim3 grid(n_rows, dims.n_heads);
    if (bf16)
        launch_pdl(st, true, grid, dim3(64), 0, qkv_post_kernel<__nv_bfloat16>, dims, layer, rows, qkv, rope_cos, rope_sin, (__nv_bfloat16*)kcache, (__nv_bfloat16*)vcache);
    else
        launch_pdl(st, true, grid, dim3(64), 0, qkv_post_kernel<float>, dims, layer, rows, qkv, rope_cos, rope_sin, (float*)kcache, (float*)vcache);
}

void launch_attention_simt(cudaStream_t st, bool bf16, const ModelDims& dims, int layer, int n_rows,
                           const RowDesc* rows, const float* qkv, const void* kcache, const void* vcache,
                           void* attn_out, int act_layout) {
    dim3 grid(dims.n_heads, n_rows);
    const bool hd128 = dims.head_dim == 128;
    if (bf16) {
        auto K = (const __nv_bfloat16*)kcache; auto V = (const __nv_bfloat16*)vcache;
        if (hd128) launch_pdl(st, true, grid, dim3(128), 0, attention_simt_kernel<__nv_bfloat16, 4>, dims, layer, rows, qkv, K, V, attn_out, act_layout);
        else launch_pdl(st, true, grid, dim3(128), 0, attention_simt_kernel<__nv_bfloat16, 2>, dims, layer, rows, qkv, K, V, attn_out, act_layout);
    } else {
        auto K = (const float*)kcache; auto V = (const float*)vcache;
        if (hd128) launch_pdl(st, true, grid, dim3(128), 0, attention_simt_kernel<float, 4>, dims, layer, rows, qkv, K, V, attn_out, act_layout);
        else launch_pdl(st, true, grid, dim3(128), 0, attention_simt_kernel<float, 2>, dims, layer, rows, qkv, K, V, attn_out, act_layout);
    }
}

}  // namespace llma
