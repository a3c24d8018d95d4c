// Shared declarations of the LLMA engine's CUDA translation units (library-private).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace llma {

constexpr int kRowCap = 256;  // most query rows one forward pass can hold (all sequences together)
constexpr int kSeqCap = 256;  // most sequence slots of an engine

// Per-sequence decoding state, resident in device memory.  Field order is mirrored by the
// host when it reads the array back.
struct SeqState {
    int32_t active;      // 1 after prefill
    int32_t done;        // 1 once target_len (or EOS) is reached
    int32_t kv_len;      // committed K/V rows
    int32_t pending;     // newest token, not yet in the cache: input row 0 of the next step
    int32_t y_len;       // tokens emitted so far
    int32_t target_len;  // stop once y_len reaches this
    int32_t ref_len;     // reference tokens stored for this sequence
    int32_t prompt_len;
    int32_t pos, k_eff, nrows;  // plan of the step in flight
    int32_t forced_rows, forced_emit;  // replay of a given step shape (0 = decide as Algorithm 1 does)
    int32_t trace_step;                // replay: index of the next step in the trace
    int32_t k_min, k_start, k_cur;     // adaptive copy length: k_cur tokens are asked for next (0 = the step's k as given)
    int32_t last_pos, last_k_eff, last_accepted, last_emitted;
    int32_t steps, trigger_steps, copied_accepted;
};

// One forward pass works on up to kRowCap rows; these arrays say what each row is.  The rows of
// the sequences that take part are packed: sequence s owns rows seq_first[s] .. +seq_cnt[s]-1
// and rows_used is the total, so a sequence without a copy adds one row, not k+1.
struct RowDesc {
    int32_t tok[kRowCap];  // input token id
    int32_t pos[kRowCap];  // absolute position in its sequence, -1 = row unused
    int32_t seq[kRowCap];  // sequence slot
    int32_t rows_used;     // number of rows in use (0 = nothing to do); they are rows 0 .. rows_used-1
    // per sequence slot: first row, row count (0 = none) and highest position
    int32_t seq_first[kSeqCap];
    int32_t seq_cnt[kSeqCap];
    int32_t seq_maxpos[kSeqCap];
    int32_t max_pos;       // highest position among used rows (-1 if none)
};

// In-kernel timeline (measurement builds only: compile with -DLLMA_STAMPS).  Every stamped kernel gets a
// block of kStampSlots x 8 words per launch: the projections write one slot per CTA (word i = time of event
// i), the attention kernels keep (min, max) pairs over their CTAs in slot 0.  Without the flag the macros
// expand to nothing and the kernels carry no trace of them.
constexpr int kStampLaunches = 512, kStampSlots = 160;
#ifdef LLMA_STAMPS
#define LLMA_STAMP_PTR(base, launch, slot) ((base) ? (base) + ((size_t)(launch) * llma::kStampSlots + (slot)) * 8 : nullptr)
#define LLMA_STAMP(ptr, i) do { if (ptr) { unsigned long long _t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(_t)); (ptr)[i] = _t; } } while (0)
#define LLMA_STAMP_MINMAX(ptr, i) do { if (ptr) { unsigned long long _t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(_t)); atomicMin(&(ptr)[i], _t); atomicMax(&(ptr)[(i) + 1], _t); } } while (0)
#else
#define LLMA_STAMP_PTR(base, launch, slot) nullptr
#define LLMA_STAMP(ptr, i) do { } while (0)
#define LLMA_STAMP_MINMAX(ptr, i) do { } while (0)
#endif

enum : int32_t {
    kDevErrNone = 0,
    kDevErrTimeout = 1,   // a bounded wait ran out
    kDevErrCapacity = 2,  // a step would have written past max_seq
    kDevErrToken = 3,     // a token id out of range reached the device
};

struct ModelDims {
    int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
    int32_t hd_total;  // n_heads * head_dim
    int32_t max_batch, max_seq, max_ref, kp1;  // kp1 = max_k + 1 = most rows of one sequence in a decoding step
    int32_t row_cap;   // rows the activation buffers hold (multiple of 16, <= kRowCap)
    float rms_eps;
    int32_t eos_id;
};

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Activations that feed a projection are kept in one of two layouts (rc = the engine's row capacity):
//   kActF32    fp32 [rc][K]                         (CUDA-core GEMM)
//   kActSplit  bf16 [2 rc][K]: row r holds hi = bf16(v), row rc + r holds lo = bf16(v - hi), so
//              hi + lo carries 16 mantissa bits through a bf16 tensor-core product (the two halves
//              are summed in fp32)
enum ActLayout : int32_t { kActF32 = 0, kActSplit = 1 };

__device__ __forceinline__ void store_act(void* buf, int layout, int rc, int r, int64_t i, int64_t K, float v) {
    if (layout == kActF32) {
        reinterpret_cast<float*>(buf)[(int64_t)r * K + i] = v;
    } else {
        __nv_bfloat16* b = reinterpret_cast<__nv_bfloat16*>(buf);
        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
        b[(int64_t)r * K + i] = hi;
        b[(int64_t)(rc + r) * K + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
    }
}

// Every kernel of a decoding step is launched with programmatic stream serialization: it may
// start while its predecessor is still running, so it must call pdl_wait() before it touches
// anything an earlier kernel wrote (or anything an earlier kernel may still be reading).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline void launch_pdl(cudaStream_t st, bool pdl, dim3 grid, dim3 block, size_t smem, void (*kernel)(KArgs...),
                       Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// K/V cache addressing: [layer][seq][head][max_seq][head_dim]; returns the row index
__host__ __device__ __forceinline__ int64_t kv_row_index(const ModelDims& d, int layer, int seq, int head, int pos) {
    return ((((int64_t)layer * d.max_batch + seq) * d.n_heads + head) * d.max_seq + pos);
}

}  // namespace llma
