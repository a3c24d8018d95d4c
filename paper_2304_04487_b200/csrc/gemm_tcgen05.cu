// Weight-streaming GEMM on tcgen05 tensor cores: TMA -> shared-memory ring -> UMMA with the
// accumulator in tensor memory -> fused epilogue.  See gemm_tcgen05.cuh for the contract.
//
// Roles inside one CTA of 192 threads:
//   warps 0-3  epilogue: TMEM -> registers -> (cross-CTA fix-up) -> fused epilogue
//   warp  4    producer: one thread issues the TMA loads of weight and activation tiles
//   warp  5    MMA: allocates TMEM; one thread issues tcgen05.mma and the commits
// Two accumulators (2 x 64 TMEM columns: 32 for the hi half of the activations, 32 for lo) let the epilogue of one tile overlap the MMAs of
// the next.  Every wait is bounded: when one runs out the kernel raises the device error
// word, stops issuing work, lets its outstanding copies land, frees TMEM and returns.
#include <cuda.h>

#include "gemm_epilogue.cuh"
#include "gemm_tcgen05.cuh"
#include "ptx_sm100.cuh"

namespace llma {

using namespace ptx;

// Range of flat (tile, chunk) work items owned by CTA b of G.
__device__ __forceinline__ int64_t cta_begin(int64_t work, int b, int G) { return work * b / G; }

__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_ws_kernel(const GemmArgs g, const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
               const __grid_constant__ CUtensorMap map_a2, const __grid_constant__ CUtensorMap map_b) {
    const int rows_used = g.rows ? g.rows->rows_used : kMaxRows;
    if (rows_used <= 0) return;  // uniform over the grid: nothing to verify this step

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sA = base, sB = base + kGemmStages * kGemmABytes;
    float (*stage)[33] = reinterpret_cast<float (*)[33]>(gen_base + kGemmStages * (kGemmABytes + kGemmBBytes));
    uint8_t* tail = reinterpret_cast<uint8_t*>(stage) + 128 * 33 * 4;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);  // full[S], empty[S], acc_full[2], acc_empty[2]
    volatile uint32_t* sh = reinterpret_cast<volatile uint32_t*>(tail + (2 * kGemmStages + 4) * 8);
    // sh[0] = TMEM base, sh[1] = abort flag, sh[2] = epilogue broadcast word
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kGemmStages + s); };
    auto accf_bar = [&](int i) { return bar0 + 8u * (2 * kGemmStages + i); };
    auto acce_bar = [&](int i) { return bar0 + 8u * (2 * kGemmStages + 2 + i); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, b = blockIdx.x;
    const int C = g.chunks;
    const int64_t work = (int64_t)g.n_tiles * C;
    const int64_t w_beg = cta_begin(work, b, G), w_end = cta_begin(work, b + 1, G);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kGemmStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(accf_bar(i), 1); mbar_init(acce_bar(i), 4); }
        sh[1] = 0; sh[2] = 0;
        fence_mbar_init();
    }
    if (warp == 5) {
        tmem_alloc(smem_u32((const void*)&sh[0]), 2 * kGemmN);
        tmem_relinquish();
    }
    if (warp == 4 && lane == 0) {
        tma_prefetch_desc(&map_a0); tma_prefetch_desc(&map_b);
        if (g.mode == kGemmQKV) { tma_prefetch_desc(&map_a1); tma_prefetch_desc(&map_a2); }
        if (g.mode == kGemmSwiGLU) tma_prefetch_desc(&map_a1);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh[0];

    if (warp == 4) {
        // ------------------------------- producer ---------------------------------------------
        if (lane == 0) {
            int64_t it = 0;
            for (int64_t w = w_beg; w < w_end && !sh[1]; ++w, ++it) {
                const int tile = (int)(w / C), c = (int)(w - (int64_t)tile * C);
                const int s = (int)(it % kGemmStages);
                const uint32_t ph = (uint32_t)((it / kGemmStages) & 1);
                if (!mbar_wait(empty_bar(s), ph ^ 1u)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                mbar_arrive_expect_tx(full_bar(s), kGemmABytes + kGemmBBytes);
                const uint32_t dstA = sA + s * kGemmABytes;
                if (g.mode == kGemmSwiGLU) {
                    tma_load_2d(dstA, &map_a0, full_bar(s), c * 64, tile * 64);
                    tma_load_2d(dstA + kGemmABytes / 2, &map_a1, full_bar(s), c * 64, tile * 64);
                } else {
                    const int m = tile / g.tiles_per_map, r0 = (tile % g.tiles_per_map) * 128;
                    const CUtensorMap* mp = m == 0 ? &map_a0 : (m == 1 ? &map_a1 : &map_a2);
                    tma_load_2d(dstA, mp, full_bar(s), c * 64, r0);
                }
                tma_load_2d(sB + s * kGemmBBytes, &map_b, full_bar(s), c * 64, 0);
            }
            if (sh[1]) {
                // give up: let the copies already issued land before the CTA's memory goes away
                const int64_t first = it > kGemmStages ? it - kGemmStages : 0;
                for (int64_t j = first; j < it; ++j)
                    (void)mbar_wait(full_bar((int)(j % kGemmStages)), (uint32_t)((j / kGemmStages) & 1), 100000000ull);
            }
        }
    } else if (warp == 5) {
        // ------------------------------- MMA issuer ---------------------------------------------
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16_m128(kGemmN);
            int64_t it = 0;
            int seg = 0;
            for (int64_t w = w_beg; w < w_end && !sh[1]; ++seg) {
                const int tile = (int)(w / C), c0 = (int)(w - (int64_t)tile * C);
                const int c1 = (int)min((int64_t)C, c0 + (w_end - w));
                const int buf = seg & 1;
                const uint32_t use = (uint32_t)(seg >> 1);
                if (!mbar_wait(acce_bar(buf), (use & 1u) ^ 1u)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * kGemmN;
                for (int c = c0; c < c1; ++c, ++it) {
                    const int s = (int)(it % kGemmStages);
                    const uint32_t ph = (uint32_t)((it / kGemmStages) & 1);
                    if (!mbar_wait(full_bar(s), ph)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                    tc_fence_after();
                    const uint64_t da = smem_desc_sw128(sA + s * kGemmABytes);
                    const uint64_t db = smem_desc_sw128(sB + s * kGemmBBytes);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)  // 4 x K=16 slices of the 64-wide chunk: +32 bytes each
                        umma_bf16(d_tmem, da + 2 * kk, db + 2 * kk, idesc, (c > c0 || kk > 0) ? 1u : 0u);
                    umma_commit(empty_bar(s));  // stage is free once these MMAs have read it
                }
                if (sh[1]) break;
                umma_commit(accf_bar(buf));  // accumulator complete
                w += c1 - c0;
            }
        }
    } else {
        // ------------------------------- epilogue warps ------------------------------------------
        const int row = threadIdx.x;  // 0..127 = TMEM lane = output feature inside the tile
        int seg = 0;
        for (int64_t w = w_beg; w < w_end; ++seg) {
            const int tile = (int)(w / C), c0 = (int)(w - (int64_t)tile * C);
            const int c1 = (int)min((int64_t)C, c0 + (w_end - w));
            w += c1 - c0;
            const int buf = seg & 1;
            const uint32_t use = (uint32_t)(seg >> 1);
            if (threadIdx.x == 0) {
                bool ok = !sh[1] && mbar_wait(accf_bar(buf), use & 1u);
                if (!ok) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; }
                sh[2] = ok ? 1u : 0u;
            }
            epi_sync();
            const bool ok = sh[2] != 0;
            epi_sync();
            if (!ok) break;
            tc_fence_after();
            float acc[32];
            {
                float lo[32];
                const uint32_t t0 = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)buf * kGemmN;
                tmem_ld_32cols(t0, acc);
                tmem_ld_32cols(t0 + kMaxRows, lo);
#pragma unroll
                for (int j = 0; j < 32; ++j) acc[j] += lo[j];  // W * hi + W * lo
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(buf));  // MMA may overwrite this accumulator

            // ---- tiles shared by several CTAs: write the partial, the last arriver sums all ----
            const int64_t t_lo = (int64_t)tile * C, t_hi = t_lo + C;
            int b_first = (int)(t_lo * G / work);
            while (cta_begin(work, b_first + 1, G) <= t_lo) ++b_first;
            while (cta_begin(work, b_first, G) > t_lo) --b_first;
            int b_last = (int)((t_hi - 1) * G / work);
            while (cta_begin(work, b_last + 1, G) <= t_hi - 1) ++b_last;
            while (cta_begin(work, b_last, G) > t_hi - 1) --b_last;
            if (b_first != b_last) {
                const int my_slot = (w_beg >= t_lo) ? 0 : 1;  // first segment of my range, or its last
                float4* dst = reinterpret_cast<float4*>(g.ws + (((int64_t)b * 2 + my_slot) * 128 + row) * 32);
#pragma unroll
                for (int q = 0; q < 8; ++q) dst[q] = make_float4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]);
                __threadfence();
                epi_sync();
                if (threadIdx.x == 0) {
                    const int old = atomicAdd(&g.cnt[tile], 1);
                    const bool last = old == (b_last - b_first);
                    if (last) g.cnt[tile] = 0;
                    sh[2] = last ? 1u : 0u;
                }
                epi_sync();
                const bool last = sh[2] != 0;
                epi_sync();
                if (!last) continue;
                __threadfence();
#pragma unroll
                for (int j = 0; j < 32; ++j) acc[j] = 0.f;
                for (int bb = b_first; bb <= b_last; ++bb) {  // ascending k: a fixed summation order
                    const int slot = (cta_begin(work, bb, G) >= t_lo) ? 0 : 1;
                    const float4* src = reinterpret_cast<const float4*>(g.ws + (((int64_t)bb * 2 + slot) * 128 + row) * 32);
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const float4 p = __ldcg(src + q);
                        acc[4 * q] += p.x; acc[4 * q + 1] += p.y; acc[4 * q + 2] += p.z; acc[4 * q + 3] += p.w;
                    }
                }
            }
            switch (g.mode) {
                case kGemmQKV: epilogue_qkv(g, tile, row, acc, rows_used, stage); break;
                case kGemmResid: epilogue_resid(g, tile, row, acc, rows_used); break;
                case kGemmSwiGLU: epilogue_swiglu(g, tile, row, acc, rows_used, stage); break;
                case kGemmStore: epilogue_store(g, tile, row, acc, rows_used); break;
                default: epilogue_lmhead(g, tile, row, acc, rows_used, stage); break;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 2 * kGemmN);
    }
}

// ---- argmax over the per-tile partials --------------------------------------------------------
__global__ void __launch_bounds__(128) argmax_final_kernel(const RowDesc* __restrict__ rows,
                                                           const float* __restrict__ part_max,
                                                           const int32_t* __restrict__ part_idx, int n_tiles,
                                                           int32_t* __restrict__ out_tok) {
    const int r = blockIdx.x;
    if (rows->pos[r] < 0) { if (threadIdx.x == 0) out_tok[r] = -1; return; }
    float bv = -INFINITY; int bi = 0x7fffffff;
    for (int t = threadIdx.x; t < n_tiles; t += blockDim.x) {
        const float v = part_max[(int64_t)t * 32 + r]; const int i = part_idx[(int64_t)t * 32 + r];
        if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    __shared__ float sv[4]; __shared__ int si[4];
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = bv; si[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 4; ++w)
            if (sv[w] > bv || (sv[w] == bv && si[w] < bi)) { bv = sv[w]; bi = si[w]; }
        out_tok[r] = bi;
    }
}

// ---- host side ------------------------------------------------------------------------------------
int gemm_grid_for(int64_t work, int num_sms) {
    int64_t g = (work + 7) / 8;  // at least ~8 k-chunks per CTA
    if (g > num_sms) g = num_sms;
    if (g < 1) g = 1;
    return (int)g;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int make_tensor_map_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || !p) return -1;
        fn = (EncodeTiledFn)p;
    }
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return (int)fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

cudaError_t init_gemm_tcgen05() {
    return cudaFuncSetAttribute(gemm_ws_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGemmSmemBytes);
}

void launch_gemm_tcgen05(cudaStream_t st, int grid, const GemmArgs& args, const CUtensorMap& a0, const CUtensorMap& a1,
                         const CUtensorMap& a2, const CUtensorMap& b) {
    gemm_ws_kernel<<<grid, kGemmThreads, kGemmSmemBytes, st>>>(args, a0, a1, a2, b);
}

void launch_argmax_final(cudaStream_t st, const RowDesc* rows, const float* part_max, const int32_t* part_idx,
                         int32_t n_tiles, int32_t* out_tok) {
    argmax_final_kernel<<<kMaxRows, 128, 0, st>>>(rows, part_max, part_idx, n_tiles, out_tok);
}

}  // namespace llma
