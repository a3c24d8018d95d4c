// Measurement aid: how long the tensor core is busy with one tcgen05.mma of the shape the projection kernels
// issue (M 128, K 16, bf16 inputs, fp32 accumulator in TMEM), as a function of N, of the number of TMEM regions
// the MMAs are dealt over, and of the commits issued in between.  One CTA, operands (zeros) resident in shared
// memory, one issuing thread: the figure is the instruction rate that bounds gemm_ws_kernel and gemm_wide_kernel.
#include <cuda_runtime.h>

#include "engine.h"
#include "ptx_sm100.cuh"

namespace llma {

using namespace ptx;

constexpr int kMbA = 4 * 16384;  // four weight-tile-sized A operands, taken in turn
constexpr int kMbB = 256 * 128;  // 256 rows of one 64-wide k-chunk

__global__ void __launch_bounds__(128) microbench_mma_kernel(int n, int regions, int groups, int commits,
                                                             unsigned long long* out_ns, int32_t* err) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sA = base, sB = base + kMbA;
    uint64_t* bar = reinterpret_cast<uint64_t*>(gbase + kMbA + kMbB);  // [0] completion, [1] target of the commits in between
    volatile uint32_t* sh = reinterpret_cast<volatile uint32_t*>(bar + 2);
    for (int i = threadIdx.x; i < (kMbA + kMbB) / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(gbase)[i] = 0;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(bar), 1);
        mbar_init(smem_u32(bar + 1), (1u << 20) - 1u);  // never completes: the commits only have to be issued
        fence_mbar_init();
    }
    fence_proxy_async_shared();
    __syncthreads();
    if (threadIdx.x < 32) { tmem_alloc(smem_u32((const void*)&sh[0]), 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh[0];
    if (threadIdx.x == 0) {
        const uint32_t idesc = idesc_bf16_m128((uint32_t)n);
        const uint64_t db = smem_desc_sw128(sB);
        const unsigned long long t0 = globaltimer_ns();
        int issued = 0;
        for (int it = 0; it < groups; ++it) {  // a group = the four k-slices of one 64-wide chunk
            const uint64_t da = smem_desc_sw128(sA + (uint32_t)(it & 3) * 16384u);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk, ++issued)
                umma_bf16(tmem + (uint32_t)((issued % regions) * n), da + 2 * kk, db + 2 * kk, idesc, issued >= regions ? 1u : 0u);
            for (int c = 0; c < commits; ++c) umma_commit(smem_u32(bar + 1));
        }
        umma_commit(smem_u32(bar));
        const bool ok = mbar_wait(smem_u32(bar), 0);  // bounded
        const unsigned long long t1 = globaltimer_ns();
        if (!ok) atomicExch(err, kDevErrTimeout);
        *out_ns = t1 - t0;
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

}  // namespace llma

using namespace llma;

extern "C" int llma_microbench_mma(int32_t n, int32_t regions, int32_t groups, int32_t commits_per_group,
                                   double* ns_per_mma) {
    if (!ns_per_mma) return LLMA_ERR_NULL;
    if (n < 16 || n > 256 || n % 16 || regions < 1 || regions * n > 512 || groups < 1 || groups > (1 << 16) ||
        commits_per_group < 0 || commits_per_group > 4)
        return LLMA_ERR_ARG;
    int dev = 0;
    cudaDeviceProp prop;
    CU_TRY(cudaGetDevice(&dev));
    CU_TRY(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return LLMA_ERR_CONFIG;
    const int smem = kMbA + kMbB + 1024 + 64;
    CU_TRY(cudaFuncSetAttribute(microbench_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    unsigned long long* d_ns = nullptr;
    int32_t* d_err = nullptr;
    CU_TRY(cudaMalloc(&d_ns, sizeof(*d_ns)));
    if (cudaMalloc(&d_err, sizeof(*d_err)) != cudaSuccess) { cudaFree(d_ns); return LLMA_ERR_CUDA; }
    int rc = LLMA_OK;
    unsigned long long ns = 0;
    int32_t err = 0;
    for (int rep = 0; rep < 2 && rc == LLMA_OK; ++rep) {  // the second launch is the one reported
        if (cudaMemset(d_err, 0, sizeof(*d_err)) != cudaSuccess) { rc = LLMA_ERR_CUDA; break; }
        microbench_mma_kernel<<<1, 128, smem>>>(n, regions, groups, commits_per_group, d_ns, d_err);
        if (cudaDeviceSynchronize() != cudaSuccess) { rc = LLMA_ERR_CUDA; break; }
        if (cudaMemcpy(&ns, d_ns, sizeof(ns), cudaMemcpyDeviceToHost) != cudaSuccess ||
            cudaMemcpy(&err, d_err, sizeof(err), cudaMemcpyDeviceToHost) != cudaSuccess) { rc = LLMA_ERR_CUDA; break; }
        if (err) rc = LLMA_ERR_DEVICE_TIMEOUT;
    }
    cudaFree(d_ns); cudaFree(d_err);
    if (rc == LLMA_OK) *ns_per_mma = (double)ns / (4.0 * groups);
    return rc;
}
