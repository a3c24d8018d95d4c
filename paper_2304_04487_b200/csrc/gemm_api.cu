// Stand-alone entry point for the weight-streaming GEMM (tests and micro-benchmarks).
#include <cstring>

#include "engine.h"

using namespace llma;

namespace llma {
// Shared by the stand-alone entry points: TMA descriptors and one launch.  `a` is the split
// activation buffer [64][k_in] (hi rows, then lo rows).
int gemm_rows32_launch(const void* W, const void* a, float* out, int32_t n_out, int32_t k_in, float* ws,
                       int32_t* dev_err, int grid, cudaStream_t st) {
    CUtensorMap ma;
    if (make_tensor_map_bf16_chunks(&ma, W, (uint64_t)n_out, (uint64_t)k_in, 128) != 0) return LLMA_ERR_ARG;
    GemmArgs g;
    std::memset(&g, 0, sizeof(g));
    g.mode = kGemmStore; g.n_out = n_out; g.n_tiles = (n_out + 127) / 128; g.chunks = k_in / 64;
    g.tiles_per_map = g.n_tiles; g.rows = nullptr; g.ws = ws; g.dev_err = dev_err;
    g.out_f32 = out; g.ld = n_out; g.act = a;
    g.rc = 32; g.nr = 32;  // the operand is [64][k_in]: 32 rows, then their low halves
    launch_gemm_tcgen05(st, grid, false, g, ma, ma, ma);
    CU_TRY(cudaGetLastError());
    return LLMA_OK;
}
}  // namespace llma

extern "C" int llma_gemm_rows32_bf16(const void* W, const void* a, float* out, int32_t n_out, int32_t k_in,
                                     void* cuda_stream) {
    if (!W || !a || !out) return LLMA_ERR_NULL;
    if (n_out < 1 || k_in < 64 || k_in % 64) return LLMA_ERR_ARG;
    int dev = 0;
    cudaDeviceProp prop;
    CU_TRY(cudaGetDevice(&dev));
    CU_TRY(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return LLMA_ERR_CONFIG;
    CU_TRY(init_gemm_tcgen05());
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int n_tiles = (n_out + 127) / 128;
    const int grid = gemm_grid_for((int64_t)n_tiles * (k_in / 64), prop.multiProcessorCount);
    float* ws = nullptr;
    int32_t* cnt = nullptr;   // one error word (after n_tiles unused words)
    __nv_bfloat16* a2 = nullptr;  // the kernel's operand: rows 0..31 = a, rows 32..63 = 0 (no low half)
    const size_t a_bytes = (size_t)32 * k_in * sizeof(__nv_bfloat16);
    CU_TRY(cudaMalloc((void**)&ws, (size_t)grid * 2 * 128 * 32 * sizeof(float)));
    cudaError_t ce = cudaMalloc((void**)&cnt, ((size_t)n_tiles + 1) * sizeof(int32_t));
    if (ce == cudaSuccess) ce = cudaMalloc((void**)&a2, 2 * a_bytes);
    if (ce != cudaSuccess) { cudaFree(ws); cudaFree(cnt); llma::note_cuda_error(ce); return LLMA_ERR_CUDA; }
    int rc = LLMA_OK;
    int32_t err = 0;
    ce = cudaMemsetAsync(cnt, 0, ((size_t)n_tiles + 1) * sizeof(int32_t), st);
    if (ce == cudaSuccess) ce = cudaMemsetAsync(ws, 0xFF, (size_t)grid * 2 * 128 * 32 * sizeof(float), st);  // hand-over slots empty
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(a2, a, a_bytes, cudaMemcpyDeviceToDevice, st);
    if (ce == cudaSuccess) ce = cudaMemsetAsync((char*)a2 + a_bytes, 0, a_bytes, st);
    if (ce == cudaSuccess) rc = gemm_rows32_launch(W, a2, out, n_out, k_in, ws, cnt + n_tiles, grid, st);
    if (ce == cudaSuccess && rc == LLMA_OK)
        ce = cudaMemcpyAsync(&err, cnt + n_tiles, sizeof(int32_t), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    cudaFree(ws);
    cudaFree(cnt);
    cudaFree(a2);
    if (ce != cudaSuccess) { llma::note_cuda_error(ce); return LLMA_ERR_CUDA; }
    if (rc) return rc;
    return err == kDevErrNone ? LLMA_OK : LLMA_ERR_DEVICE_TIMEOUT;
}
