// llma_gemm_rows32_bf16_noalloc: the stand-alone projection GEMM for callers that must not
// allocate.  Its partial tiles (handed between CTAs), error word and the 64-row operand
// staging live in one file-scope __device__ array instead of cudaMalloc'ed memory.
#include <cstring>
#include <mutex>

#include "engine.h"

using namespace llma;

namespace llma {
int gemm_rows32_launch(const void* W, const void* a, float* out, int32_t n_out, int32_t k_in, float* ws,
                       int32_t* dev_err, int grid, cudaStream_t st);
}

namespace {

constexpr int kMaxGrid = 160;        // CTAs whose partial tiles fit (a B200 has 148 SMs)
constexpr int kMaxTiles = 2048;      // n_out <= 262144
constexpr int kMaxK = 16384;         // k_in limit of the operand staging
constexpr size_t kWsBytes = (size_t)kMaxGrid * 2 * 128 * 32 * sizeof(float);      // 5,242,880
constexpr size_t kCntBytes = ((size_t)(kMaxTiles + 1) * sizeof(int32_t) + 255) / 256 * 256;
constexpr size_t kOperandBytes = (size_t)64 * kMaxK * sizeof(__nv_bfloat16);     // 2,097,152
constexpr size_t kScratchBytes = kWsBytes + kCntBytes + kOperandBytes;            // about 7.0 MiB

// Every GPU that loads this library holds this array until the process exits.  In host
// code the name below is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_ptr[kMaxDevices] = {nullptr};
int g_sm_count[kMaxDevices] = {0};

}  // namespace

extern "C" int llma_gemm_rows32_bf16_noalloc(const void* W, const void* a, float* out, int32_t n_out, int32_t k_in,
                                             void* cuda_stream) {
    if (!W || !a || !out) return LLMA_ERR_NULL;
    if (n_out < 1 || k_in < 64 || k_in % 64) return LLMA_ERR_ARG;
    const int n_tiles = (n_out + 127) / 128;
    if (n_tiles > kMaxTiles || k_in > kMaxK) return LLMA_ERR_CAPACITY;  // beyond the fixed scratch
    int dev = 0;
    CU_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return LLMA_ERR_CONFIG;
    unsigned char* base = nullptr;
    int sms = 0;
    {
        // one-time set-up per device, with that device current: resolve the array's device address
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_scratch_ptr[dev]) {
            int major = 0, count = 0;
            CU_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
            CU_TRY(cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev));
            if (major != 10) return LLMA_ERR_CONFIG;
            CU_TRY(init_gemm_tcgen05());
            unsigned char* p = nullptr;
            CU_TRY(cudaGetSymbolAddress((void**)&p, g_noalloc_scratch));
            g_sm_count[dev] = count;
            g_scratch_ptr[dev] = p;
        }
        base = g_scratch_ptr[dev];
        sms = g_sm_count[dev];
    }
    float* ws = reinterpret_cast<float*>(base);
    int32_t* cnt = reinterpret_cast<int32_t*>(base + kWsBytes);
    __nv_bfloat16* operand = reinterpret_cast<__nv_bfloat16*>(base + kWsBytes + kCntBytes);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int grid = gemm_grid_for((int64_t)n_tiles * (k_in / 64), sms);
    if (grid > kMaxGrid) grid = kMaxGrid;
    const size_t a_bytes = (size_t)32 * k_in * sizeof(__nv_bfloat16);
    // the array keeps the previous call's contents: the error word must start at
    // zero, and the low half of the operand must be zero (this entry point takes plain bf16 rows)
    CU_TRY(cudaMemsetAsync(cnt, 0, ((size_t)n_tiles + 1) * sizeof(int32_t), st));
    // the partial-tile hand-over slots must read as empty (all-ones words) when the kernel starts
    CU_TRY(cudaMemsetAsync(ws, 0xFF, (size_t)grid * 2 * 128 * 32 * sizeof(float), st));
    CU_TRY(cudaMemcpyAsync(operand, a, a_bytes, cudaMemcpyDeviceToDevice, st));
    CU_TRY(cudaMemsetAsync(reinterpret_cast<char*>(operand) + a_bytes, 0, a_bytes, st));
    int rc = gemm_rows32_launch(W, operand, out, n_out, k_in, ws, cnt + n_tiles, grid, st);
    if (rc) return rc;
    int32_t err = 0;
    CU_TRY(cudaMemcpyAsync(&err, cnt + n_tiles, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    return err == kDevErrNone ? LLMA_OK : LLMA_ERR_DEVICE_TIMEOUT;
}
