// CUDA-core kernels of the decoder forward: RMSNorm, small-M GEMM, SiLU gating, argmax.
// They serve fp32 models (where tensor cores would break the 1e-4 logit tolerance) and are
// the plain cross-check of the tensor-core path for bf16 models.
//
// Every output element is computed by a fixed sequence of operations that depends only on
// its own row's data and on the matrix shape -- never on how many rows the step has.  That
// is what makes a (k+1)-row verification step bit-identical to k+1 one-row greedy steps.
#include "kernels.h"

namespace llma {

// ---- RMSNorm -----------------------------------------------------------------------------
__global__ void __launch_bounds__(256) rmsnorm_kernel(const RowDesc* __restrict__ rows, const float* __restrict__ x,
                                                      const float* __restrict__ g, void* __restrict__ out, int layout,
                                                      int rc, int d, float eps) {
    pdl_trigger();
    pdl_wait();
    const int r = blockIdx.x;
    const float* xr = x + (int64_t)r * d;
    if (rows->pos[r] < 0) {
        for (int i = threadIdx.x; i < d; i += blockDim.x) store_act(out, layout, rc, r, i, d, 0.f);
        return;
    }
    float ss = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) ss += xr[i] * xr[i];
    __shared__ float red[8];
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < 8; ++w) tot += red[w];  // fixed order
    const float inv = rsqrtf(tot / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += blockDim.x) store_act(out, layout, rc, r, i, d, xr[i] * inv * g[i]);
}

// ---- small-M GEMM: one warp per output feature --------------------------------------------
// out[r, n] = sum_k W[n, k] * a[r, k].  Lane l owns k in {l*V + i*32*V + v}; the 32 lane
// partials are combined by an xor butterfly.  V = elements per 16-byte load.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    __device__ static void load(const float* p, float (&v)[4]) {
        float4 t = *reinterpret_cast<const float4*>(p);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static void load(const __nv_bfloat16* p, float (&v)[8]) {
        uint4 t = *reinterpret_cast<const uint4*>(p);
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

template <typename T, int RB>  // RB rows handled per pass over the weight row
__global__ void __launch_bounds__(256) gemm_simt_kernel(const RowDesc* __restrict__ rows, const T* __restrict__ W,
                                                        const float* __restrict__ a, float* __restrict__ out, int n_out,
                                                        int k_in, int ld_out, int accumulate) {
    pdl_trigger();
    pdl_wait();
    constexpr int V = Vec16<T>::N;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= n_out) return;
    const int rows_used = rows->rows_used;
    const T* wrow = W + (int64_t)warp * k_in;
    for (int r0 = 0; r0 < rows_used; r0 += RB) {
        float acc[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r) acc[r] = 0.f;
        for (int kk = lane * V; kk < k_in; kk += 32 * V) {
            float wv[V];
            Vec16<T>::load(wrow + kk, wv);
#pragma unroll
            for (int r = 0; r < RB; ++r) {
                if (r0 + r < rows_used) {
                    const float* ap = a + (int64_t)(r0 + r) * k_in + kk;
#pragma unroll
                    for (int v4 = 0; v4 < V; v4 += 4) {
                        float av[4];
                        Vec16<float>::load(ap + v4, av);
#pragma unroll
                        for (int v = 0; v < 4; ++v) acc[r] = fmaf(wv[v4 + v], av[v], acc[r]);
                    }
                }
            }
        }
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            float s = acc[r];
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane == 0 && r0 + r < rows_used) {
                float* dst = out + (int64_t)(r0 + r) * ld_out + warp;
                *dst = accumulate ? (*dst + s) : s;
            }
        }
    }
}

// ---- SiLU gating ----------------------------------------------------------------------------
__global__ void silu_mul_kernel(const RowDesc* __restrict__ rows, const float* __restrict__ gate_up,
                                float* __restrict__ h, int d_ffn) {
    pdl_trigger();
    pdl_wait();
    const int r = blockIdx.y;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= d_ffn) return;
    float v = 0.f;
    if (r < rows->rows_used) {
        const float g = gate_up[(int64_t)r * 2 * d_ffn + i];
        const float u = gate_up[(int64_t)r * 2 * d_ffn + d_ffn + i];
        v = g / (1.f + expf(-g)) * u;
    }
    h[(int64_t)r * d_ffn + i] = v;
}

// ---- per-row argmax, lowest index on ties --------------------------------------------------
__global__ void __launch_bounds__(256) argmax_kernel(const RowDesc* __restrict__ rows, const float* __restrict__ logits,
                                                     int vocab, int32_t* __restrict__ out_tok) {
    pdl_trigger();
    pdl_wait();
    const int r = blockIdx.x;
    if (rows->pos[r] < 0) { if (threadIdx.x == 0) out_tok[r] = -1; return; }
    const float* lr = logits + (int64_t)r * vocab;
    float bv = -INFINITY; int bi = 0x7fffffff;
    for (int i = threadIdx.x; i < vocab; i += blockDim.x) {
        float v = lr[i];
        if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    __shared__ float sv[8]; __shared__ int si[8];
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = bv; si[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w)
            if (sv[w] > bv || (sv[w] == bv && si[w] < bi)) { bv = sv[w]; bi = si[w]; }
        out_tok[r] = bi;
    }
}

// ---- launchers -------------------------------------------------------------------------------
void launch_rmsnorm(cudaStream_t st, int act_layout, int n_rows, int rc, const RowDesc* rows, const float* x,
                    const float* g, void* x_hat, int32_t d, float eps) {
    launch_pdl(st, true, dim3(n_rows), dim3(256), 0, rmsnorm_kernel, rows, x, g, x_hat, act_layout, rc, d, eps);
}

void launch_gemm_simt(cudaStream_t st, bool bf16, const RowDesc* rows, const void* W, const float* a, float* out,
                      int32_t n_out, int32_t k_in, int32_t ld_out, bool accumulate) {
    const int blocks = (n_out + 7) / 8;
    if (bf16)
        launch_pdl(st, true, dim3(blocks), dim3(256), 0, gemm_simt_kernel<__nv_bfloat16, 8>, rows, (const __nv_bfloat16*)W, a, out, n_out, k_in, ld_out, accumulate ? 1 : 0);
    else
        launch_pdl(st, true, dim3(blocks), dim3(256), 0, gemm_simt_kernel<float, 8>, rows, (const float*)W, a, out, n_out, k_in, ld_out, accumulate ? 1 : 0);
}

void launch_silu_mul(cudaStream_t st, int n_rows, const RowDesc* rows, const float* gate_up, float* h, int32_t d_ffn) {
    dim3 grid((d_ffn + 255) / 256, n_rows);
    launch_pdl(st, true, grid, dim3(256), 0, silu_mul_kernel, rows, gate_up, h, d_ffn);
}

void launch_argmax(cudaStream_t st, int n_rows, const RowDesc* rows, const float* logits, int32_t vocab, int32_t* out_tok) {
    launch_pdl(st, true, dim3(n_rows), dim3(256), 0, argmax_kernel, rows, logits, vocab, out_tok);
}

}  // namespace llma
