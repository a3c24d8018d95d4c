// Weight-streaming GEMM for up to 256 activation rows (batched decoding steps, prompt passes).
// Same contract, work split and fused epilogues as gemm_ws_kernel (see gemm_tcgen05.cuh); what differs:
//   * the activation tiles are large enough for TMA to pay: a second producer thread streams them
//     through a ring of their own (one slot = nr rows x 64 columns of ONE bf16 term, hi or lo); both terms
//     are accumulated into the same TMEM columns;
//   * a ring stage of weights holds 256 rows (two 128-row tiles, or 128 gate + 128 up rows), multiplied by the same
//     activation tile into two accumulators: every activation byte fetched from L2 serves twice the weights;
//   * MMA N = the rows in use rounded up to 16 (a run-time field of the instruction descriptor);
//   * the epilogue walks a finished 128 x nr accumulator in blocks of 32 rows.
//
// Roles inside one CTA of 224 threads:
//   warps 0-3  epilogue: TMEM -> registers -> (cross-CTA fix-up) -> fused epilogue, block by block
//   warp  4    one thread issues the TMA loads of the weight tiles (they depend on no earlier kernel)
//   warp  5    MMA: allocates TMEM; one thread issues tcgen05.mma and the commits
//   warp  6    one thread issues the TMA loads of the activation tiles (after the dependency wait)
//
// Every wait is bounded: when one runs out the kernel raises the device error word, stops
// issuing work, lets its outstanding copies land, frees TMEM and returns.
#include <cuda.h>

#include "gemm_epilogue.cuh"
#include "gemm_tcgen05.cuh"
#include "ptx_sm100.cuh"

namespace llma {

using namespace ptx;

constexpr size_t kWideStageBytes = 128 * 33 * 4;
constexpr size_t kWideTailBytes = 5120;  // barriers, flags, per-row scales, reduction scratch, row positions and slots
constexpr uint32_t kWideABytes = 2 * kGemmABytes;  // a stage of weights: 256 rows x one 64-wide k-chunk

template <int MODE>
__global__ void __launch_bounds__(kGemmWideThreads, 1)
gemm_wide_kernel(const GemmArgs g, const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
                 const __grid_constant__ CUtensorMap map_a2, const __grid_constant__ CUtensorMap map_b,
                 const int SA, const int SB, const uint32_t tmem_cols) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
    const int nr = g.nr;
    constexpr int NT = 2;  // bf16 terms of the activation operand: hi, lo
    const uint32_t b_slot = (uint32_t)nr * 128u;
    const uint32_t sA = base, sB = base + (uint32_t)SA * kWideABytes;
    uint8_t* after = gen_base + (size_t)SA * kWideABytes + (size_t)SB * b_slot;
    float (*stage)[33] = reinterpret_cast<float (*)[33]>(after);
    float (*stage_g)[33] = stage + 128;  // gate half of a gate/up pair
    uint8_t* tail = after + 2 * kWideStageBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);  // full_a[8], empty_a[8], full_b[8], empty_b[8], acc_full[2], acc_empty[2]
    volatile uint32_t* sh = reinterpret_cast<volatile uint32_t*>(tail + 36 * 8);  // [0] TMEM base, [1] abort, [2] broadcast
    float* rscale = reinterpret_cast<float*>(tail + 36 * 8 + 16);                 // [256] per-row norm scales
    float* red_f = rscale + kRowCap;                                              // [4][32]
    int* red_i = reinterpret_cast<int*>(red_f + 128);                             // [4][32]
    int* s_pos = red_i + 128;                                                     // [256] (QKV mode)
    int* s_seq = s_pos + kRowCap;                                                 // [256]
    const uint32_t bar0 = smem_u32(bars);
    auto full_a = [&](int s) { return bar0 + 8u * s; };
    auto empty_a = [&](int s) { return bar0 + 8u * (8 + s); };
    auto full_b = [&](int s) { return bar0 + 8u * (16 + s); };
    auto empty_b = [&](int s) { return bar0 + 8u * (24 + s); };
    auto accf_bar = [&](int i) { return bar0 + 8u * (32 + i); };
    auto acce_bar = [&](int i) { return bar0 + 8u * (34 + i); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, b = blockIdx.x;
    const int C = g.chunks;
    // A work tile is 256 weight rows: two 128-row tiles of one matrix (QKV: never across two of the three
    // matrices), or, for gate/up, 128 gate rows and the same 128 up rows (g.n_tiles counts those pairs).
    const int tpm = g.tiles_per_map;
    const int spm = MODE == kGemmSwiGLU ? tpm : (tpm + 1) / 2;          // work tiles per matrix
    const int n_super = MODE == kGemmSwiGLU ? g.n_tiles : (g.n_tiles / tpm) * spm;
    const int64_t work = (int64_t)n_super * C;
    const int64_t w_beg = cta_begin(work, b, G), w_end = cta_begin(work, b + 1, G);
    const int n_buf = 4 * nr <= 512 ? 2 : 1;  // accumulator sets (of two accumulators of nr columns) that fit TMEM
    // the 128-row tile that half h of work tile S is (an index the epilogues understand), or -1 if past its matrix
    auto sub_tile = [&](int S, int h) {
        if (MODE == kGemmSwiGLU) return S;
        const int m = S / spm, lt = 2 * (S - m * spm) + h;
        return lt < tpm ? m * tpm + lt : -1;
    };

    grid_launch_dependents();  // the next kernel may begin its own prologue now
    if (threadIdx.x == 0) {
        for (int s = 0; s < 8; ++s) {
            mbar_init(full_a(s), 1); mbar_init(empty_a(s), 1); mbar_init(full_b(s), 1); mbar_init(empty_b(s), 1);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(accf_bar(i), 1); mbar_init(acce_bar(i), 4); }
        sh[1] = 0; sh[2] = 0;
        fence_mbar_init();
    }
    if (warp == 5) {
        tmem_alloc(smem_u32((const void*)&sh[0]), tmem_cols);
        tmem_relinquish();
    }
    if (warp == 4 && lane == 0) {
        tma_prefetch_desc(&map_a0);
        if (MODE == kGemmQKV) { tma_prefetch_desc(&map_a1); tma_prefetch_desc(&map_a2); }
        if (MODE == kGemmSwiGLU) tma_prefetch_desc(&map_a1);
    }
    if (warp == 6 && lane == 0) tma_prefetch_desc(&map_b);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh[0];

    if (warp == 4) {
        // ------------------------------- weight producer -----------------------------------------
        if (lane == 0) {
            int64_t it = 0;
            for (int64_t w = w_beg; w < w_end && !sh[1]; ++w, ++it) {
                const int s = (int)(it % SA);
                const uint32_t ph = (uint32_t)((it / SA) & 1);
                if (it >= SA && !mbar_wait(empty_a(s), ph ^ 1u)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                mbar_arrive_expect_tx(full_a(s), kWideABytes);
                const int S = (int)(w / C), c = (int)(w - (int64_t)S * C);
                const uint32_t dstA = sA + s * kWideABytes;
                if (MODE == kGemmSwiGLU) {
                    tma_load_2d(dstA, &map_a0, full_a(s), c * 64, S * 128);
                    tma_load_2d(dstA + kGemmABytes, &map_a1, full_a(s), c * 64, S * 128);
                } else {  // one copy of 256 rows (rows past the matrix arrive as zeros)
                    const int m = S / spm, r0 = (S - m * spm) * 256;
                    const CUtensorMap* mp = m == 0 ? &map_a0 : (m == 1 ? &map_a1 : &map_a2);
                    tma_load_2d(dstA, mp, full_a(s), c * 64, r0);
                }
            }
            if (sh[1]) {  // give up: let the copies already issued land before the CTA's memory goes away
                const int64_t first = it > SA ? it - SA : 0;
                for (int64_t j = first; j < it; ++j)
                    (void)mbar_wait(full_a((int)(j % SA)), (uint32_t)((j / SA) & 1), 100000000ull);
            }
        }
    } else if (warp == 6) {
        // ------------------------------- activation producer ---------------------------------------
        if (lane == 0) {
            grid_dependency_wait();  // activations are written by the kernel before this one
            int64_t it = 0;          // counts (item, term) pairs
            for (int64_t w = w_beg; w < w_end && !sh[1]; ++w) {
                const int c = (int)(w % C);
                for (int t = 0; t < NT; ++t, ++it) {
                    const int s = (int)(it % SB);
                    const uint32_t ph = (uint32_t)((it / SB) & 1);
                    if (it >= SB && !mbar_wait(empty_b(s), ph ^ 1u)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                    mbar_arrive_expect_tx(full_b(s), b_slot);
                    tma_load_2d(sB + (uint32_t)s * b_slot, &map_b, full_b(s), c * 64, t * g.rc);
                }
                if (sh[1]) break;
            }
            if (sh[1]) {
                const int64_t first = it > SB ? it - SB : 0;
                for (int64_t j = first; j < it; ++j)
                    (void)mbar_wait(full_b((int)(j % SB)), (uint32_t)((j / SB) & 1), 100000000ull);
            }
        }
    } else if (warp == 5) {
        // ------------------------------- MMA issuer ---------------------------------------------
        if (lane == 0) {
            grid_dependency_wait();  // the count of rows in use comes from the planning kernel
            int rows_used = g.rows ? __ldcg(&g.rows->rows_used) : nr;
            rows_used = max(1, min(rows_used, nr));
            const uint32_t idesc = idesc_bf16_m128((uint32_t)((rows_used + 15) & ~15));
            int64_t ia = 0, ib = 0;
            int seg = 0;
            for (int64_t w = w_beg; w < w_end && !sh[1]; ++seg) {
                const int S = (int)(w / C), c0 = (int)(w - (int64_t)S * C);
                const int c1 = (int)min((int64_t)C, c0 + (w_end - w));
                const int buf = seg % n_buf;
                const uint32_t use = (uint32_t)(seg / n_buf);
                if (!mbar_wait(acce_bar(buf), (use & 1u) ^ 1u)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 2) * (uint32_t)nr;  // the set's two accumulators
                for (int c = c0; c < c1 && !sh[1]; ++c, ++ia) {
                    const int s = (int)(ia % SA);
                    if (!mbar_wait(full_a(s), (uint32_t)((ia / SA) & 1))) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                    for (int t = 0; t < NT; ++t, ++ib) {
                        const int sb = (int)(ib % SB);
                        if (!mbar_wait(full_b(sb), (uint32_t)((ib / SB) & 1))) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                        tc_fence_after();
                        const uint64_t db = smem_desc_sw128(sB + (uint32_t)sb * b_slot);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {  // the two 128-row halves of the weight stage share the activation tile
                            const uint64_t da = smem_desc_sw128(sA + s * kWideABytes + h * kGemmABytes);
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk)  // 4 x K=16 slices of the 64-wide chunk: +32 bytes each
                                umma_bf16(d_tmem + (uint32_t)h * (uint32_t)nr, da + 2 * kk, db + 2 * kk, idesc,
                                          (c > c0 || kk > 0 || t > 0) ? 1u : 0u);
                        }
                        umma_commit(empty_b(sb));  // slot is free once these MMAs have read it
                    }
                    if (sh[1]) break;
                    umma_commit(empty_a(s));
                }
                if (sh[1]) break;
                umma_commit(accf_bar(buf));  // accumulators complete
                w += c1 - c0;
            }
        }
    } else {
        // ------------------------------- epilogue warps ------------------------------------------
        grid_dependency_wait();  // everything below reads or writes what earlier kernels produced
        const int rows_used = g.rows ? min(g.rows->rows_used, nr) : nr;
        const int nblk = (rows_used + 31) >> 5;
        const int row = threadIdx.x;  // 0..127 = TMEM lane = output feature inside the tile
        if (g.ss_in) {  // folded RMSNorm: one scale per activation row, tiles summed in ascending order
            for (int r = row; r < rows_used; r += 128) {
                float ssum = 0.f;
                int t = 0;
                for (; t + 8 <= g.ss_tiles; t += 8) {  // eight loads in flight
                    float v[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) v[u] = __ldcg(&g.ss_in[(int64_t)(t + u) * g.rc + r]);
#pragma unroll
                    for (int u = 0; u < 8; ++u) ssum += v[u];
                }
                for (; t < g.ss_tiles; ++t) ssum += __ldcg(&g.ss_in[(int64_t)t * g.rc + r]);
                rscale[r] = rsqrtf(ssum / (float)g.norm_dim + g.norm_eps);
            }
        }
        if (MODE == kGemmQKV) {  // the rows' positions and sequence slots, read once per CTA
            for (int r = row; r < rows_used; r += 128) {
                s_pos[r] = __ldcg(&g.rows->pos[r]);
                s_seq[r] = __ldcg(&g.rows->seq[r]);
            }
        }
        epi_sync();
        const float xnone[kXPre] = {};
        // a 32-row block of one accumulator goes to shared memory (scaled by the folded RMSNorm)
        auto stage_block = [&](float (*dst)[33], int jb, const float (&acc)[32]) {
            if (g.ss_in) {
#pragma unroll
                for (int j = 0; j < 32; ++j) dst[row][j] = acc[j] * rscale[min(jb + j, kRowCap - 1)];
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) dst[row][j] = acc[j];
            }
        };
        // the fused epilogue of a staged block (gate/up: of the pair of staged blocks)
        auto run_block = [&](int tile, int rb) {
            const int jb = rb * 32, nj = min(32, rows_used - jb);
            epi_sync();
            if constexpr (MODE == kGemmQKV) epilogue_qkv(g, tile, row, jb, nj, stage, s_pos, s_seq, nullptr);
            else if constexpr (MODE == kGemmResid) epilogue_resid<false>(g, tile, row, jb, nj, stage, red_f, xnone);
            else if constexpr (MODE == kGemmSwiGLU) epilogue_swiglu_pair(g, tile, row, jb, nj, stage_g, stage);
            else if constexpr (MODE == kGemmStore) epilogue_store(g, tile, row, jb, nj, stage);
            else epilogue_lmhead(g, tile, row, jb, nj, stage, red_f, red_i);
            epi_sync();  // the staging area is rewritten by the next block
        };
        // Tiles cut by a range boundary (see gemm_ws_kernel): the CTA that holds a work tile's FIRST chunks owns
        // it and completes it at the end of its range; every other CTA of the tile hands its two partial
        // accumulators over through its slot pair of the workspace (all-ones words while empty).  The slots are
        // laid out for the engine's row capacity whatever nr is, so that prompt passes and decoding steps agree on them.
        constexpr uint32_t kEmpty = 0xFFFFFFFFu;
        const int qn = g.rc >> 2;
        bool aborted = false;
        int seg = 0;
        for (int64_t w = w_beg; w < w_end; ++seg) {
            const int S = (int)(w / C), c0 = (int)(w - (int64_t)S * C);
            const int c1 = (int)min((int64_t)C, c0 + (w_end - w));
            w += c1 - c0;
            const int buf = seg % n_buf;
            const uint32_t use = (uint32_t)(seg / n_buf);
            if (threadIdx.x == 0) {
                bool ok = !sh[1] && mbar_wait(accf_bar(buf), use & 1u);
                if (!ok) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; }
                sh[2] = ok ? 1u : 0u;
            }
            epi_sync();
            const bool ok = sh[2] != 0;
            epi_sync();
            if (!ok) { aborted = true; break; }
            tc_fence_after();
            const int64_t t_lo = (int64_t)S * C, t_hi = t_lo + C;
            const bool hand_over = w_beg > t_lo;            // another CTA holds the tile's first chunks
            const bool owner = !hand_over && w_end < t_hi;  // this one does, and others hold the rest
            int b_last = b;
            if (owner) {
                b_last = (int)((t_hi - 1) * G / work);
                while (cta_begin(work, b_last + 1, G) <= t_hi - 1) ++b_last;
                while (cta_begin(work, b_last, G) > t_hi - 1) --b_last;
            }
            const unsigned long long give_up = globaltimer_ns() + 2000000000ull;
            const uint32_t t0 = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * 2) * (uint32_t)nr;
            for (int rb = 0; rb < nblk; ++rb) {
                const int jb = rb * 32;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int tile = sub_tile(S, h);
                    if (tile < 0) continue;  // past the matrix (uniform over the CTA)
                    float acc[32];
                    tmem_ld_32cols(t0 + (uint32_t)h * (uint32_t)nr + (uint32_t)rb * 32u, acc);
                    if (hand_over) {
                        float4* dst = ws_slot(g.ws, qn, b, h, row) + (int64_t)rb * 8 * 128;
#pragma unroll
                        for (int q = 0; q < 8; ++q)  // only the columns of rows in use travel
                            if (jb + 4 * q < rows_used) dst[q * 128] = make_float4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]);
                        continue;
                    }
                    for (int bb = b + 1; bb <= b_last; ++bb) {  // owner: the later CTAs' partials in ascending k
                        float4* src = ws_slot(g.ws, qn, bb, h, row) + (int64_t)rb * 8 * 128;
                        float4 p[8];
                        bool valid;
                        do {
                            valid = true;
#pragma unroll
                            for (int q = 0; q < 8; ++q)
                                if (jb + 4 * q < rows_used) p[q] = ld_poll_f4(src + q * 128);
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                if (jb + 4 * q < rows_used) {
                                    valid = valid && __float_as_uint(p[q].x) != kEmpty;
                                    if (jb + 4 * q + 1 < rows_used) valid = valid && __float_as_uint(p[q].y) != kEmpty;
                                    if (jb + 4 * q + 2 < rows_used) valid = valid && __float_as_uint(p[q].z) != kEmpty;
                                    if (jb + 4 * q + 3 < rows_used) valid = valid && __float_as_uint(p[q].w) != kEmpty;
                                }
                            }
                            if (!valid && globaltimer_ns() > give_up) { atomicExch(g.dev_err, kDevErrTimeout); break; }
                        } while (!valid);
                        const float e = __uint_as_float(kEmpty);
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            if (jb + 4 * q < rows_used) {
                                src[q * 128] = make_float4(e, e, e, e);  // empty again for the next projection
                                acc[4 * q] += p[q].x; acc[4 * q + 1] += p[q].y; acc[4 * q + 2] += p[q].z; acc[4 * q + 3] += p[q].w;
                            }
                        }
                    }
                    if (MODE == kGemmSwiGLU) {
                        stage_block(h == 0 ? stage_g : stage, jb, acc);
                        if (h == 1) run_block(tile, rb);
                    } else {
                        stage_block(stage, jb, acc);
                        run_block(tile, rb);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(buf));  // MMA may overwrite this accumulator set
        }
        (void)aborted;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// ---- host side ------------------------------------------------------------------------------------
GemmWideCfg gemm_wide_cfg(int nr) {
    GemmWideCfg c;
    c.b_slot = (uint32_t)nr * 128u;
    const size_t budget = (size_t)227 * 1024 - 1024 - 2 * kWideStageBytes - kWideTailBytes;
    // three weight stages first, then as many activation tiles as fit (at least three), then more weight stages
    c.sa = 3;
    c.sb = (int)((budget - (size_t)c.sa * kWideABytes) / c.b_slot);
    if (c.sb < 3) { c.sa = 2; c.sb = (int)((budget - (size_t)c.sa * kWideABytes) / c.b_slot); }
    if (c.sb > 8) c.sb = 8;
    c.sa = (int)((budget - (size_t)c.sb * c.b_slot) / kWideABytes);
    if (c.sa > 6) c.sa = 6;
    uint32_t cols = 32;
    const uint32_t need = 4u * (uint32_t)nr <= 512u ? 4u * (uint32_t)nr : 2u * (uint32_t)nr;  // two sets of two accumulators, or one
    while (cols < need) cols <<= 1;
    c.tmem_cols = cols;
    c.smem_bytes = 1024 + (size_t)c.sa * kWideABytes + (size_t)c.sb * c.b_slot + 2 * kWideStageBytes + kWideTailBytes;
    if (c.smem_bytes < 120 * 1024) c.smem_bytes = 120 * 1024;  // one CTA per SM, as for the narrow kernel
    return c;
}

template <int MODE>
static cudaError_t wide_opt_in() {
    return cudaFuncSetAttribute(gemm_wide_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

cudaError_t init_gemm_wide() {
    cudaError_t e;
    if ((e = wide_opt_in<kGemmQKV>()) != cudaSuccess) return e;
    if ((e = wide_opt_in<kGemmResid>()) != cudaSuccess) return e;
    if ((e = wide_opt_in<kGemmSwiGLU>()) != cudaSuccess) return e;
    if ((e = wide_opt_in<kGemmLmHead>()) != cudaSuccess) return e;
    return wide_opt_in<kGemmStore>();
}

void launch_gemm_wide(cudaStream_t st, int grid, bool pdl, const GemmArgs& args, const CUtensorMap& a0,
                      const CUtensorMap& a1, const CUtensorMap& a2, const CUtensorMap& map_b) {
    const GemmWideCfg c = gemm_wide_cfg(args.nr);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kGemmWideThreads);
    cfg.dynamicSmemBytes = c.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    const int sa = c.sa, sb = c.sb;
    const uint32_t cols = c.tmem_cols;
    switch (args.mode) {
        case kGemmQKV: cudaLaunchKernelEx(&cfg, gemm_wide_kernel<kGemmQKV>, args, a0, a1, a2, map_b, sa, sb, cols); break;
        case kGemmResid: cudaLaunchKernelEx(&cfg, gemm_wide_kernel<kGemmResid>, args, a0, a1, a2, map_b, sa, sb, cols); break;
        case kGemmSwiGLU: cudaLaunchKernelEx(&cfg, gemm_wide_kernel<kGemmSwiGLU>, args, a0, a1, a2, map_b, sa, sb, cols); break;
        case kGemmLmHead: cudaLaunchKernelEx(&cfg, gemm_wide_kernel<kGemmLmHead>, args, a0, a1, a2, map_b, sa, sb, cols); break;
        default: cudaLaunchKernelEx(&cfg, gemm_wide_kernel<kGemmStore>, args, a0, a1, a2, map_b, sa, sb, cols); break;
    }
}

}  // namespace llma
