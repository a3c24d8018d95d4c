// Weight-streaming GEMM on tcgen05 tensor cores: TMA -> shared-memory ring -> UMMA with the
// accumulator in tensor memory -> fused epilogue.  See gemm_tcgen05.cuh for the contract.
//
// Roles inside one CTA of 320 threads:
//   warps 0-3  epilogue: TMEM -> registers -> (cross-CTA fix-up) -> fused epilogue
//   warp  4    producer: one thread issues the TMA loads of the weight tiles
//   warp  5    MMA: allocates TMEM; one thread issues tcgen05.mma and the commits
//   warps 6-9  activation loaders: they take turns filling the activation tile of a ring stage with
//              plain loads and swizzled shared-memory stores
// Two accumulators in TMEM let the epilogue of one tile overlap the MMAs of the next.
//
// Programmatic dependent launch: the kernel lets its successor start at once, and itself
// starts streaming WEIGHT tiles (which no earlier kernel writes) without waiting for its
// predecessor; only the activation loaders and the epilogue warps wait for it.  So the prologue and pipeline fill of one projection overlap the tail of the
// kernel before it.
//
// Every wait is bounded: when one runs out the kernel raises the device error word, stops
// issuing work, lets its outstanding copies land, frees TMEM and returns.
#include <cuda.h>

#include "gemm_epilogue.cuh"
#include "gemm_tcgen05.cuh"
#include "ptx_sm100.cuh"

namespace llma {

using namespace ptx;

// NR = activation rows: 16 or 32.  The hi and lo halves of the activations are the MMA's N = 2 NR columns
// (one MMA per k-slice: an MMA this narrow costs the same issue time whatever its N, so two N = NR MMAs into
// one accumulator measured 15 % slower); the epilogue adds the two halves.  MODE = GemmMode: one kernel per fused
// epilogue, so that each carries only the code it runs (the end of a launch is instruction-fetch-bound).
template <int NR, int MODE>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_ws_kernel(const GemmArgs g, const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
               const __grid_constant__ CUtensorMap map_a2) {
    constexpr int KC = kGemmKC;             // 64-wide k-chunks per ring stage (one TMA copy)
    using Cfg = GemmCfg<NR>;
    constexpr int NT = 2;                   // bf16 terms of the activation operand: hi, lo
    constexpr uint32_t kTmemCols = 4 * NR;  // two accumulators of 2 NR columns
    constexpr int S = Cfg::kStages;
    constexpr uint32_t kABytes = Cfg::kABytes, kBBytes = Cfg::kBBytes, kBTile = Cfg::kBTile;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sA = base, sB = base + S * kABytes;
    float (*stage)[33] = reinterpret_cast<float (*)[33]>(gen_base + S * (kABytes + kBBytes));
    uint8_t* tail = reinterpret_cast<uint8_t*>(stage) + 128 * 33 * 4;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);  // full[S], empty[S], acc_full[2], acc_empty[2]
    volatile uint32_t* sh = reinterpret_cast<volatile uint32_t*>(tail + (2 * S + 4) * 8);
    float* rscale = reinterpret_cast<float*>(tail + (2 * S + 4) * 8 + 16);  // [32] per-row norm scales
    float* red_f = rscale + 32;                                             // [4][32] reduction scratch
    int* red_i = reinterpret_cast<int*>(red_f + 128);                       // [4][32]
    float2* rope_s = reinterpret_cast<float2*>(tail + 1536);                // [32][head_dim / 2] (QKV mode)
    // sh[0] = TMEM base, sh[1] = abort flag, sh[2] = epilogue broadcast word
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
    auto accf_bar = [&](int i) { return bar0 + 8u * (2 * S + i); };
    auto acce_bar = [&](int i) { return bar0 + 8u * (2 * S + 2 + i); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, b = blockIdx.x;
    const int C = (g.chunks + KC - 1) / KC;  // work items (ring stages) per tile
    const int64_t work = (int64_t)g.n_tiles * C;
    const int64_t w_beg = cta_begin(work, b, G), w_end = cta_begin(work, b + 1, G);

    grid_launch_dependents();  // the next kernel may begin its own prologue now
    // timeline events: 0 CTA start, 1 dependency released, 2 first stage ready, 3 last MMA issued, 4 last accumulator ready, 5 CTA end
    [[maybe_unused]] unsigned long long* stp = LLMA_STAMP_PTR(g.stamps, g.launch_id, blockIdx.x);
    if (threadIdx.x == 0) LLMA_STAMP(stp, 0);
    if (threadIdx.x == 0) {
        // a stage is full once its weight tile has landed (producer's expect_tx) and the loader warps of its
        // KC activation tiles have arrived
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1 + KC); mbar_init(empty_bar(s), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(accf_bar(i), 1); mbar_init(acce_bar(i), 4); }
        sh[1] = 0; sh[2] = 0;
        fence_mbar_init();
    }
    if (warp == 5) {
        tmem_alloc(smem_u32((const void*)&sh[0]), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 4 && lane == 0) {
        tma_prefetch_desc(&map_a0);
        if (MODE == kGemmQKV) { tma_prefetch_desc(&map_a1); tma_prefetch_desc(&map_a2); }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh[0];

    if (warp == 4) {
        // ------------------------------- producer ---------------------------------------------
        if (lane == 0) {
            auto load_a = [&](int64_t w, int s) {
                const int tile = (int)(w / C), c = (int)(w - (int64_t)tile * C);
                const uint32_t dstA = sA + s * kABytes;
                // chunks 2c and 2c+1 of the tile in one copy (a chunk past the matrix arrives as zeros)
                if (MODE == kGemmSwiGLU) {  // 64 rows of each of the two matrices per chunk
                    tma_load_4d(dstA, &map_a0, full_bar(s), 0, tile * 64, 0, c * KC);
                } else {
                    const int m = tile / g.tiles_per_map, r0 = (tile % g.tiles_per_map) * 128;
                    const CUtensorMap* mp = m == 0 ? &map_a0 : (m == 1 ? &map_a1 : &map_a2);
                    tma_load_3d(dstA, mp, full_bar(s), 0, r0, c * KC);
                }
            };
            // weights are written by no kernel of the step: the whole range streams without waiting for
            // the predecessor (the MMAs wait for the activation loaders, which do)
            int64_t it = 0;
            for (int64_t w = w_beg; w < w_end && !sh[1]; ++w, ++it) {
                const int s = (int)(it % S);
                const uint32_t ph = (uint32_t)((it / S) & 1);
                if (it >= S && !mbar_wait(empty_bar(s), ph ^ 1u)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                mbar_arrive_expect_tx(full_bar(s), kABytes);
                load_a(w, s);
            }
            if (sh[1]) {
                // give up: let the copies already issued land before the CTA's memory goes away
                const int64_t first = it > S ? it - S : 0;
                for (int64_t j = first; j < it; ++j)
                    (void)mbar_wait(full_bar((int)(j % S)), (uint32_t)((j / S) & 1), 100000000ull);
            }
        }
    } else if (warp == 5) {
        // ------------------------------- MMA issuer ---------------------------------------------
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16_m128(2 * NR);
            int64_t it = 0;
            int seg = 0;
            for (int64_t w = w_beg; w < w_end && !sh[1]; ++seg) {
                const int tile = (int)(w / C), c0 = (int)(w - (int64_t)tile * C);
                const int c1 = (int)min((int64_t)C, c0 + (w_end - w));
                const int buf = seg & 1;
                const uint32_t use = (uint32_t)(seg >> 1);
                if (!mbar_wait(acce_bar(buf), (use & 1u) ^ 1u)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * (2 * NR);
                for (int c = c0; c < c1; ++c, ++it) {
                    const int s = (int)(it % S);
                    const uint32_t ph = (uint32_t)((it / S) & 1);
                    if (!mbar_wait(full_bar(s), ph)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                    if (it == 0) LLMA_STAMP(stp, 2);
                    tc_fence_after();
#pragma unroll
                    for (int h = 0; h < KC; ++h) {  // the stage's k-chunks: a weight tile and an activation tile each
                        const uint64_t da = smem_desc_sw128(sA + s * kABytes + h * kGemmABytes);
                        const uint64_t db = smem_desc_sw128(sB + s * kBBytes + h * kBTile);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)  // 4 x K=16 slices of the 64-wide chunk: +32 bytes each
                            umma_bf16(d_tmem, da + 2 * kk, db + 2 * kk, idesc, (c > c0 || h > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(empty_bar(s));  // stage is free once these MMAs have read it
                }
                if (sh[1]) break;
                umma_commit(accf_bar(buf));  // accumulator complete
                LLMA_STAMP(stp, 3);
                w += c1 - c0;
            }
        }
    } else if (warp >= 6) {
        // ------------------------------- activation loaders ----------------------------------------
        // Tile layout in shared memory (what the MMA's K-major, 128-byte
        // swizzled descriptor reads): row r = 0..NT*NR-1 (NR rows per term) at r * 128 bytes, its
        // 16-byte unit j stored at position j ^ (r & 7).  Rows past those in use are left as they are:
        // their columns of the accumulator are never read.
        constexpr int NW = 4;  // loader warps: warp 6 + i takes activation tiles i, i + NW, ... (KC tiles per stage)
        const int sw = warp - 6;
        grid_dependency_wait();  // activations are written by the kernel before this one
        const int rows_used = g.rows ? min(__ldcg(&g.rows->rows_used), NR) : NR;
        const int64_t n_sub = (w_end - w_beg) * KC;
        const int64_t ld_bytes = (int64_t)g.chunks * 128;  // one activation row: k_in bf16
        const char* act = reinterpret_cast<const char*>(g.act);
        constexpr int kUnits = NT * NR * 8 / 32;    // 16-byte units per lane
        if constexpr (NR == 32) {
            // Thirty-two rows: the tile goes from global to shared memory by asynchronous 16-byte copies, with no
            // registers in between (a register copy of the next tile costs 64 of them, and with those the CTA
            // leaves no room on the SM for a CTA of the attention kernel).  A copy is issued as soon as its
            // stage is free and handed to the MMA warp when it has landed.
            auto issue = [&](int64_t q, int row_limit) {
                const int64_t it = q / KC;
                const int chunk = (int)((w_beg + it) % C) * KC + (int)(q % KC);
                const bool inside = chunk < g.chunks;
                const uint32_t dst0 = sB + (uint32_t)(it % S) * kBBytes + (uint32_t)(q % KC) * kBTile;
#pragma unroll
                for (int u = 0; u < kUnits; ++u) {
                    const int unit = u * 32 + lane, r = unit >> 3, j = unit & 7;
                    const int t = r / NR, rr = r - t * NR;
                    const uint32_t dst = dst0 + (uint32_t)r * 128 + (uint32_t)((j ^ (r & 7)) << 4);
                    if (rr < row_limit) {
                        if (inside) cp_async_16(dst, act + (t * g.rc + rr) * ld_bytes + (int64_t)chunk * 128 + j * 16);
                        else st_shared_v4(dst, make_uint4(0u, 0u, 0u, 0u));  // past the matrix: zeros
                    }
                }
                cp_async_commit();
            };
            for (int64_t q = sw; q < n_sub && !sh[1]; q += NW) {
                const int64_t it = q / KC;
                if (it >= S) {
                    bool ok = true;
                    if (lane == 0) ok = mbar_wait(empty_bar((int)(it % S)), (uint32_t)((it / S) & 1) ^ 1u);
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { if (lane == 0) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; } break; }
                }
                issue(q, q == sw ? NR : rows_used);  // first tile: every row, the count of rows is still on its way
                cp_async_wait<0>();                  // L2 latency: shorter than that of the weight copy issued at the same moment
                fence_proxy_async_shared();
                __syncwarp();
                if (lane == 0) mbar_arrive(full_bar((int)(it % S)));
            }
        } else {
        // rows of the next tile are requested before waiting for its stage to come free, so the
        // latency of the loads hides behind the MMAs of the tiles in between
        uint4 v[kUnits];
        auto fetch = [&](int64_t q, int row_limit) {
            const int64_t it = q / KC;
            const int chunk = (int)((w_beg + it) % C) * KC + (int)(q % KC);  // 64-wide chunk of the activations
            const bool inside = chunk < g.chunks;                            // past the matrix: zeros
#pragma unroll
            for (int u = 0; u < kUnits; ++u) {
                const int unit = u * 32 + lane, r = unit >> 3, j = unit & 7;
                const int t = r / NR, rr = r - t * NR;                // term, row inside it
                const int src_row = t * g.rc + rr;                    // term t starts at row t * rc
                v[u] = make_uint4(0u, 0u, 0u, 0u);
                if (rr < row_limit && inside)
                    v[u] = __ldcg(reinterpret_cast<const uint4*>(act + src_row * ld_bytes + (int64_t)chunk * 128 + j * 16));
            }
        };
        if (sw < n_sub) fetch(sw, NR);  // every row: the count of rows in use is still on its way
        for (int64_t q = sw; q < n_sub && !sh[1]; q += NW) {
            const int64_t it = q / KC;
            const int h = (int)(q % KC);
            const int st = (int)(it % S);
            const uint32_t ph = (uint32_t)((it / S) & 1);
            if (it >= S) {
                bool ok = true;
                if (lane == 0) ok = mbar_wait(empty_bar(st), ph ^ 1u);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { if (lane == 0) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; } break; }
            }
#pragma unroll
            for (int u = 0; u < kUnits; ++u) {
                const int unit = u * 32 + lane, r = unit >> 3, j = unit & 7;
                const int rr = r % NR;
                if (rr < rows_used)
                    st_shared_v4(sB + st * kBBytes + h * kBTile + (uint32_t)r * 128 + (uint32_t)((j ^ (r & 7)) << 4), v[u]);
            }
            fence_proxy_async_shared();  // make the stores visible to the tensor core's reads
            __syncwarp();
            if (lane == 0) mbar_arrive(full_bar(st));
            if (q + NW < n_sub) fetch(q + NW, rows_used);
        }
        }
    } else {
        // ------------------------------- epilogue warps ------------------------------------------
        grid_dependency_wait();  // everything below reads or writes what earlier kernels produced
        if (threadIdx.x == 0) LLMA_STAMP(stp, 1);
        const int rows_used = g.rows ? min(g.rows->rows_used, NR) : NR;
        const int row = threadIdx.x;  // 0..127 = TMEM lane = output feature inside the tile
        if (g.ss_in && row < NR) {  // folded RMSNorm: one scale per activation row, tiles summed in ascending order
            float ssum = 0.f;
            int t = 0;
            for (; t + 8 <= g.ss_tiles; t += 8) {  // eight loads in flight
                float v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = __ldcg(&g.ss_in[(int64_t)(t + u) * g.rc + row]);
#pragma unroll
                for (int u = 0; u < 8; ++u) ssum += v[u];
            }
            for (; t < g.ss_tiles; ++t) ssum += __ldcg(&g.ss_in[(int64_t)t * g.rc + row]);
            rscale[row] = rsqrtf(ssum / (float)g.norm_dim + g.norm_eps);
        }
        if (MODE == kGemmQKV) {  // the rows' positions and sequence slots, read once per CTA
            if (row < 32) red_i[row] = __ldcg(&g.rows->pos[row]);
            else if (row < 64) red_i[row] = __ldcg(&g.rows->seq[row - 32]);
        }
        epi_sync();
        if (MODE == kGemmQKV) {
            // rotary factors of every row in use, once per CTA: the tile epilogues then read shared memory only
            const int half = g.dims.head_dim >> 1;
            for (int idx = row; idx < rows_used * half; idx += 128) {
                const int j = idx / half, fi = idx - j * half;
                const int pos = red_i[j];
                float2 cs = make_float2(1.f, 0.f);
                if (pos >= 0) cs = make_float2(__ldg(&g.rope_cos[(int64_t)pos * half + fi]), __ldg(&g.rope_sin[(int64_t)pos * half + fi]));
                rope_s[j * half + fi] = cs;
            }
            epi_sync();
        }
        constexpr bool kPrefetchX = true;
        // residual rows of a tile: requested early, so their latency hides behind the accumulator wait
        // and the cross-CTA sum (only the tile's owner ever writes them, in its epilogue)
        auto prefetch_x = [&](int tile, float (&xpre)[kXPre]) {
            if (kPrefetchX && MODE == kGemmResid) {
                const int col = tile * 128 + row;
#pragma unroll
                for (int u = 0; u < kXPre - 1; ++u)
                    xpre[u] = (col < g.n_out && u < rows_used) ? __ldcg(&g.out_f32[(int64_t)u * g.ld + col]) : 0.f;
                xpre[kXPre - 1] = (col < g.n_out && g.xs_out) ? __ldg(&g.gain_next[col]) : 0.f;  // the next norm's gain
            }
        };
        // stage the tile in shared memory (scaled by the folded RMSNorm), then the fused epilogue
        auto finish_tile = [&](int tile, float (&acc)[32], const float (&xpre)[kXPre]) {
            if (g.ss_in) {
#pragma unroll
                for (int j = 0; j < NR; ++j) stage[row][j] = acc[j] * rscale[j];
            } else {
#pragma unroll
                for (int j = 0; j < NR; ++j) stage[row][j] = acc[j];
            }
            epi_sync();
            if constexpr (MODE == kGemmQKV) epilogue_qkv(g, tile, row, 0, rows_used, stage, red_i, red_i + 32, rope_s);
            else if constexpr (MODE == kGemmResid) epilogue_resid<kPrefetchX>(g, tile, row, 0, rows_used, stage, red_f, xpre);
            else if constexpr (MODE == kGemmSwiGLU) epilogue_swiglu(g, tile, row, 0, rows_used, stage);
            else if constexpr (MODE == kGemmStore) epilogue_store(g, tile, row, 0, rows_used, stage);
            else epilogue_lmhead(g, tile, row, 0, rows_used, stage, red_f, red_i);
        };
        // Tiles cut by a range boundary.  The CTA whose range holds the tile's FIRST chunks owns it: that is
        // the last thing it works on, so it completes the tile at once.  Every other CTA of the tile hands its
        // partial over through its slot of the workspace, whose words hold the bit pattern kEmpty (a NaN no
        // arithmetic here produces) while nothing has been handed over: the owner polls the words it needs
        // until none is kEmpty, adds the partials in ascending k order (its own first), and puts kEmpty back.
        // No fence, counter or second pass.  The CTA that holds a tile's LAST chunks works on them first, long
        // before the owner asks: a tile cut in two costs its owner no wait at all; only CTAs whose whole range
        // lies inside one tile finish together with the owner.
        constexpr uint32_t kEmpty = 0xFFFFFFFFu;
        bool aborted = false;
        int seg = 0;
        for (int64_t w = w_beg; w < w_end; ++seg) {
            const int tile = (int)(w / C), c0 = (int)(w - (int64_t)tile * C);
            const int c1 = (int)min((int64_t)C, c0 + (w_end - w));
            w += c1 - c0;
            const int buf = seg & 1;
            const uint32_t use = (uint32_t)(seg >> 1);
            float xpre[kXPre];
            prefetch_x(tile, xpre);
            if (threadIdx.x == 0) {
                bool ok = !sh[1] && mbar_wait(accf_bar(buf), use & 1u);
                if (!ok) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; }
                sh[2] = ok ? 1u : 0u;
            }
            epi_sync();
            const bool ok = sh[2] != 0;
            epi_sync();
            if (!ok) { aborted = true; break; }
            if (threadIdx.x == 0) LLMA_STAMP(stp, 4);
            tc_fence_after();
            float acc[32];
            {
                const uint32_t t0 = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)buf * (2 * NR);
                if (NR == 32) {
                    tmem_ld_32cols(t0, acc);
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {  // W * hi + W * lo, the low term sixteen columns at a time
                        float lo[16];
                        tmem_ld_16cols(t0 + 32 + 16 * hf, lo);
#pragma unroll
                        for (int j = 0; j < 16; ++j) acc[16 * hf + j] += lo[j];
                    }
                } else {
                    tmem_ld_32cols(t0, acc);  // columns 0..15 hi, 16..31 lo
#pragma unroll
                    for (int j = 0; j < 16; ++j) { acc[j] += acc[16 + j]; acc[16 + j] = 0.f; }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(buf));  // MMA may overwrite this accumulator

            const int64_t t_lo = (int64_t)tile * C, t_hi = t_lo + C;
            if (w_beg > t_lo) {  // another CTA holds the tile's first chunks: hand this partial over to it
                float4* dst = ws_slot(g.ws, NR / 4, b, 1, row);
#pragma unroll
                for (int q = 0; q < NR / 4; ++q)  // only the columns of rows in use travel
                    if (4 * q < rows_used) dst[q * 128] = make_float4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]);
                continue;
            }
            if (w_end < t_hi) {  // this CTA owns the tile; the CTAs after it hold the rest of its chunks
                int b_last = (int)((t_hi - 1) * G / work);
                while (cta_begin(work, b_last + 1, G) <= t_hi - 1) ++b_last;
                while (cta_begin(work, b_last, G) > t_hi - 1) --b_last;
                const unsigned long long give_up = globaltimer_ns() + 2000000000ull;
                constexpr int kBatch = NR == 32 ? 1 : 2;  // partials requested together (registers)
                for (int bb = b + 1; bb <= b_last; bb += kBatch) {  // ascending k: a fixed summation order
                    float4 p[kBatch][NR / 4];
                    bool valid;
                    do {
                        valid = true;
#pragma unroll
                        for (int u = 0; u < kBatch; ++u) {
                            if (bb + u <= b_last) {
                                const float4* src = ws_slot(g.ws, NR / 4, bb + u, 1, row);
#pragma unroll
                                for (int q = 0; q < NR / 4; ++q)
                                    if (4 * q < rows_used) p[u][q] = ld_poll_f4(src + q * 128);
                            }
                        }
#pragma unroll
                        for (int u = 0; u < kBatch; ++u) {
                            if (bb + u <= b_last) {
#pragma unroll
                                for (int q = 0; q < NR / 4; ++q) {
                                    if (4 * q < rows_used) {
                                        valid = valid && __float_as_uint(p[u][q].x) != kEmpty;
                                        if (4 * q + 1 < rows_used) valid = valid && __float_as_uint(p[u][q].y) != kEmpty;
                                        if (4 * q + 2 < rows_used) valid = valid && __float_as_uint(p[u][q].z) != kEmpty;
                                        if (4 * q + 3 < rows_used) valid = valid && __float_as_uint(p[u][q].w) != kEmpty;
                                    }
                                }
                            }
                        }
                        if (!valid && globaltimer_ns() > give_up) { atomicExch(g.dev_err, kDevErrTimeout); break; }
                    } while (!valid);
                    const float e = __uint_as_float(kEmpty);
#pragma unroll
                    for (int u = 0; u < kBatch; ++u) {
                        if (bb + u <= b_last) {
                            float4* src = ws_slot(g.ws, NR / 4, bb + u, 1, row);
#pragma unroll
                            for (int q = 0; q < NR / 4; ++q) {
                                if (4 * q < rows_used) {
                                    src[q * 128] = make_float4(e, e, e, e);  // empty again for the next projection
                                    acc[4 * q] += p[u][q].x; acc[4 * q + 1] += p[u][q].y;
                                    acc[4 * q + 2] += p[u][q].z; acc[4 * q + 3] += p[u][q].w;
                                }
                            }
                        }
                    }
                }
            }
            if (threadIdx.x == 0) LLMA_STAMP(stp, 6);  // partials summed: the tile's epilogue begins
            finish_tile(tile, acc, xpre);
        }
        (void)aborted;
        if (threadIdx.x == 0) LLMA_STAMP(stp, 5);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
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

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || !p) return nullptr;
        fn = (EncodeTiledFn)p;
    }
    return fn;
}

int make_tensor_map_bf16_chunks(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || cols % 64) return -1;
    const cuuint64_t dims[3] = {64, rows, cols / 64};
    const cuuint64_t strides[2] = {cols * 2, 128};
    const cuuint32_t box[3] = {64, box_rows, 2};
    const cuuint32_t estr[3] = {1, 1, 1};
    return (int)fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

int make_tensor_map_bf16_pair(CUtensorMap* out, const void* base0, const void* base1, uint64_t rows, uint64_t cols,
                              int* swapped) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || cols % 64 || base0 == base1) return -1;
    const uintptr_t p0 = (uintptr_t)base0, p1 = (uintptr_t)base1;
    *swapped = p1 < p0 ? 1 : 0;
    const uintptr_t lo = *swapped ? p1 : p0, diff = *swapped ? p0 - p1 : p1 - p0;
    if (diff % 16 || diff >= (1ull << 40) || diff < rows * cols * 2) return -1;
    const cuuint64_t dims[4] = {64, rows, 2, cols / 64};
    const cuuint64_t strides[3] = {cols * 2, (cuuint64_t)diff, 128};
    const cuuint32_t box[4] = {64, 64, 2, 2};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return (int)fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, reinterpret_cast<void*>(lo), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

int make_tensor_map_bf16_terms(CUtensorMap* out, const void* base, uint64_t rc, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || box_rows > 256) return -1;
    const cuuint64_t dims[3] = {cols, rc, 2};
    const cuuint64_t strides[2] = {cols * 2, rc * cols * 2};
    const cuuint32_t box[3] = {64, box_rows, 2};
    const cuuint32_t estr[3] = {1, 1, 1};
    return (int)fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

int make_tensor_map_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return -1;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return (int)fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

template <int NR, int MODE>
static cudaError_t opt_in() {
    return cudaFuncSetAttribute(gemm_ws_kernel<NR, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)GemmCfg<NR>::kSmemBytes);
}
template <int NR>
static cudaError_t opt_in_all() {
    cudaError_t e;
    if ((e = opt_in<NR, kGemmQKV>()) != cudaSuccess) return e;
    if ((e = opt_in<NR, kGemmResid>()) != cudaSuccess) return e;
    if ((e = opt_in<NR, kGemmSwiGLU>()) != cudaSuccess) return e;
    if ((e = opt_in<NR, kGemmLmHead>()) != cudaSuccess) return e;
    return opt_in<NR, kGemmStore>();
}

cudaError_t init_gemm_tcgen05() {
    cudaError_t e = opt_in_all<16>();
    if (e != cudaSuccess) return e;
    return opt_in_all<32>();
}

template <int NR>
static void launch_mode(cudaLaunchConfig_t* cfg, const GemmArgs& args, const CUtensorMap& a0, const CUtensorMap& a1,
                        const CUtensorMap& a2) {
    switch (args.mode) {
        case kGemmQKV: cudaLaunchKernelEx(cfg, gemm_ws_kernel<NR, kGemmQKV>, args, a0, a1, a2); break;
        case kGemmResid: cudaLaunchKernelEx(cfg, gemm_ws_kernel<NR, kGemmResid>, args, a0, a1, a2); break;
        case kGemmSwiGLU: cudaLaunchKernelEx(cfg, gemm_ws_kernel<NR, kGemmSwiGLU>, args, a0, a1, a2); break;
        case kGemmLmHead: cudaLaunchKernelEx(cfg, gemm_ws_kernel<NR, kGemmLmHead>, args, a0, a1, a2); break;
        default: cudaLaunchKernelEx(cfg, gemm_ws_kernel<NR, kGemmStore>, args, a0, a1, a2); break;
    }
}

void launch_gemm_tcgen05(cudaStream_t st, int grid, bool pdl, const GemmArgs& args, const CUtensorMap& a0,
                         const CUtensorMap& a1, const CUtensorMap& a2) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = args.nr == 16 ? GemmCfg<16>::kSmemBytes : GemmCfg<32>::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    if (args.nr == 16) launch_mode<16>(&cfg, args, a0, a1, a2);
    else launch_mode<32>(&cfg, args, a0, a1, a2);
}

}  // namespace llma
