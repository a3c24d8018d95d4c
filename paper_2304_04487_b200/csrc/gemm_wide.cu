// Weight-streaming GEMM for up to 256 activation rows (batched decoding steps, prompt passes).
// Same contract, work split and fused epilogues as gemm_ws_kernel (see gemm_tcgen05.cuh); what differs:
//   * the activation tiles are large enough for TMA to pay: a ring stage holds the weight tile of one 64-wide
//     k-chunk and, behind it, the chunk's activation tile (the nr hi rows, then the nr lo rows, fetched by one
//     copy through a 3-D view of the split buffer); two producer warps fill the two halves of a stage, because
//     only the activations have to wait for the kernel before;
//   * an accumulator has 2 nr columns [hi | lo], summed by the epilogue: up to 128 rows one MMA of N = 2 nr per
//     k-slice and two accumulators in turn; beyond, two MMAs per k-slice (N = the rows in use rounded up to 16,
//     a run-time field of the instruction descriptor) and a single accumulator.  An MMA of this shape (M 128,
//     K 16) occupies the tensor core for about 81 ns whatever its N (measured for N = 16 .. 256, alone and dealt
//     over several accumulators) and a commit costs the issuing thread another 45 ns, so the number of MMAs and
//     commits per weight tile is what bounds the kernel: 4 + 1 up to 128 rows (0.37 us per 16 KB, the HBM rate),
//     8 + 1 beyond;
//   * the rows a copy brings (nr: 32, 64, 128 or the launch's capacity) are chosen per step from the rows in use;
//   * the epilogue walks a finished 128 x nr accumulator in blocks of 32 rows; tiles cut by a range boundary
//     are summed and finished block by block by all the CTAs that share them.
//
// Roles inside one CTA of 224 threads:
//   warps 0-3  epilogue: TMEM -> registers -> workspace (cut tiles) or fused epilogue, block by block; then the
//              blocks of cut tiles dealt to this CTA
//   warp  4    one or two lanes issue the TMA loads of the weight tiles (they depend on no earlier kernel)
//   warp  5    MMA: allocates TMEM; one thread issues tcgen05.mma and the commits
//   warp  6    one or two lanes issue the TMA loads of the activation tiles (after the dependency wait)
//
// Every wait is bounded: when one runs out the kernel raises the device error word, stops
// issuing work, lets its outstanding copies land, frees TMEM and returns.
#include <cuda.h>

#include <type_traits>

#include "gemm_epilogue.cuh"
#include "gemm_tcgen05.cuh"
#include "ptx_sm100.cuh"

namespace llma {

using namespace ptx;

constexpr size_t kWideStageBytes = 128 * 33 * 4;
constexpr size_t kWideTailBytes = 5120;  // barriers, flags, per-row scales, reduction scratch, row positions and slots

template <int MODE>
__global__ void __launch_bounds__(kGemmWideThreads, 1)
gemm_wide_kernel(const GemmArgs g, const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
                 const __grid_constant__ CUtensorMap map_a2, const __grid_constant__ CUtensorMap map_b0,
                 const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_b2,
                 const __grid_constant__ CUtensorMap map_b3, const int SA, const uint32_t tmem_cols) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
    // g.nr is the row capacity the launch was shaped for; the rows a copy brings (nr below) are chosen per step from
    // the rows in use, by every role that needs them, once the planning kernel's count may be read
    const uint32_t stage_bytes = kGemmABytes + (uint32_t)g.nr * 256u;  // weight tile, then the largest activation tile
    auto box_index = [&](int rows_used) {
        int i = 0;
        while (i < 3 && wide_box_rows(g.nr, i) < rows_used) ++i;
        return i;
    };
    const uint32_t sA = base, sB = base + kGemmABytes;   // stage s: sA + s * stage_bytes, sB + s * stage_bytes
    uint8_t* after = gen_base + (size_t)SA * stage_bytes;
    float (*stage)[33] = reinterpret_cast<float (*)[33]>(after);
    uint8_t* tail = after + kWideStageBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);  // full[8], empty[8], (16 unused), acc_full[2], acc_empty[2]
    volatile uint32_t* sh = reinterpret_cast<volatile uint32_t*>(tail + 36 * 8);  // [0] TMEM base, [1] abort, [2] broadcast
    float* rscale = reinterpret_cast<float*>(tail + 36 * 8 + 16);                 // [256] per-row norm scales
    float* red_f = rscale + kRowCap;                                              // [4][32]
    int* red_i = reinterpret_cast<int*>(red_f + 128);                             // [4][32]
    int* s_pos = red_i + 128;                                                     // [256] (QKV mode)
    int* s_seq = s_pos + kRowCap;                                                 // [256]
    const uint32_t bar0 = smem_u32(bars);
    auto full_a = [&](int s) { return bar0 + 8u * s; };
    auto empty_a = [&](int s) { return bar0 + 8u * (8 + s); };
    auto full_b = full_a;    // both halves of a stage land on one barrier (two arrivals with their byte counts)
    auto empty_b = empty_a;  // and are released together
    auto accf_bar = [&](int i) { return bar0 + 8u * (32 + i); };
    auto acce_bar = [&](int i) { return bar0 + 8u * (34 + i); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, b = blockIdx.x;
    const int C = g.chunks;
    const int64_t work = (int64_t)g.n_tiles * C;
    const int64_t w_beg = cta_begin(work, b, G), w_end = cta_begin(work, b + 1, G);
    const int64_t n_items = w_end - w_beg;

    grid_launch_dependents();  // the next kernel may begin its own prologue now
    [[maybe_unused]] unsigned long long* stp = LLMA_STAMP_PTR(g.stamps, g.launch_id, blockIdx.x);
    if (threadIdx.x == 0) LLMA_STAMP(stp, 0);
    if (threadIdx.x == 0) {
        for (int s = 0; s < 8; ++s) {
            mbar_init(full_a(s), 2); mbar_init(empty_a(s), 1);
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
    if (warp == 6 && lane == 0) { tma_prefetch_desc(&map_b0); tma_prefetch_desc(&map_b1); tma_prefetch_desc(&map_b2); tma_prefetch_desc(&map_b3); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh[0];

    // One thread gets a TMA copy under way about every 0.5 us, whatever the copy's size (measured: 16 KB boxes from one
    // thread stream 31 GB/s per CTA, from two threads 59, from four 95, L2-resident), so each half of a stage is
    // filled by two lanes in turn where the ring has four stages or more (its depth is then even: see gemm_wide_cfg).
    // Stage, parity, tile and chunk of a lane's next item are kept as running counters: divisions by run-time
    // values would cost these threads as much as the copies.
    const int kP = SA >= 4 ? 2 : 1;
    if (warp == 4) {
        // ------------------------------- weight producers (lane p takes items p, p + kP, ...) ------------------
        if (lane < kP) {
            int64_t it = lane;
            int tile = (int)((w_beg + lane) / C), c = (int)((w_beg + lane) - (int64_t)tile * C);
            int m = tile / g.tiles_per_map, rt = tile - m * g.tiles_per_map;  // matrix and tile inside it
            int s = lane;       // lane < kP <= SA
            uint32_t ph = 0;
            for (; it < n_items && !sh[1]; it += kP) {
                if (it >= SA && !mbar_wait(empty_a(s), ph ^ 1u)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                mbar_arrive_expect_tx(full_a(s), kGemmABytes);
                const uint32_t dstA = sA + (uint32_t)s * stage_bytes;
                if (MODE == kGemmSwiGLU) {
                    tma_load_2d(dstA, &map_a0, full_a(s), c * 64, tile * 64);
                    tma_load_2d(dstA + kGemmABytes / 2, &map_a1, full_a(s), c * 64, tile * 64);
                } else {
                    const CUtensorMap* mp = m == 0 ? &map_a0 : (m == 1 ? &map_a1 : &map_a2);
                    tma_load_2d(dstA, mp, full_a(s), c * 64, rt * 128);
                }
                c += kP;
                while (c >= C) { c -= C; ++tile; if (++rt == g.tiles_per_map) { rt = 0; ++m; } }
                s += kP;
                if (s >= SA) { s -= SA; ph ^= 1u; }
            }
            if (sh[1]) {  // give up: let this lane's copies already issued land before the CTA's memory goes away
                for (int64_t j = it - kP; j >= 0 && j > it - kP * (SA + 1); j -= kP)
                    (void)mbar_wait(full_a((int)(j % SA)), (uint32_t)((j / SA) & 1), 100000000ull);
            }
        }
    } else if (warp == 6) {
        // ------------------------------- activation producers (lane p takes items p, p + kP, ...) --------------
        if (lane < kP) {
            grid_dependency_wait();  // activations are written by the kernel before this one
            const int bi = box_index(g.rows ? min(__ldcg(&g.rows->rows_used), g.nr) : g.nr);
            const CUtensorMap* map_b = bi == 0 ? &map_b0 : (bi == 1 ? &map_b1 : (bi == 2 ? &map_b2 : &map_b3));
            const uint32_t b_slot = (uint32_t)wide_box_rows(g.nr, bi) * 256u;  // hi rows, then lo rows, of one k-chunk
            int64_t q = lane;
            int c = (int)((w_beg + lane) % C);
            int s = lane;
            uint32_t ph = 0;
            for (; q < n_items && !sh[1]; q += kP) {
                if (q >= SA && !mbar_wait(empty_b(s), ph ^ 1u)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                mbar_arrive_expect_tx(full_b(s), b_slot);
                tma_load_3d(sB + (uint32_t)s * stage_bytes, map_b, full_b(s), c * 64, 0, 0);
                c += kP;
                while (c >= C) c -= C;
                s += kP;
                if (s >= SA) { s -= SA; ph ^= 1u; }
            }
            if (sh[1]) {
                for (int64_t j = q - kP; j >= 0 && j > q - kP * (SA + 1); j -= kP)
                    (void)mbar_wait(full_b((int)(j % SA)), (uint32_t)((j / SA) & 1), 100000000ull);
            }
        }
    } else if (warp == 5) {
        // ------------------------------- MMA issuer ---------------------------------------------
        if (lane == 0) {
            grid_dependency_wait();  // the count of rows in use comes from the planning kernel
            int rows_used = g.rows ? __ldcg(&g.rows->rows_used) : g.nr;
            rows_used = max(1, min(rows_used, g.nr));
            const int nr = wide_box_rows(g.nr, box_index(rows_used));  // hi rows at 0, lo rows nr further on
            // An accumulator has 2 nr columns [hi | lo]; two accumulators take turns while they fit the 512 TMEM
            // columns, else there is one.
            const int acc_cols = 2 * nr;
            const int n_acc = 2 * acc_cols <= 512 ? 2 : 1;
            // Up to 128 rows: one MMA per k-slice over the hi and the lo rows together (N = 2 nr, columns [hi | lo]).
            // Beyond (N = 2 nr would pass the instruction's 256): two MMAs per k-slice, the hi rows into the first
            // nr columns and the lo rows into the next nr, N = the rows in use rounded up to 16.  Either way a
            // column is summed over k in the same order, so a row's result does not depend on which applies.
            const bool one_mma = 2 * nr <= 256;
            const uint32_t idesc = idesc_bf16_m128(one_mma ? (uint32_t)(2 * nr) : (uint32_t)((rows_used + 15) & ~15));
            int64_t ia = 0;
            int s = 0;            // ring stage of item ia and the parity of its use: kept by hand, a division by the
            uint32_t s_ph = 0;    // run-time ring depth would cost this thread more than a commit
            int seg = 0;
#ifdef LLMA_STAMPS
            // measurement build: time this thread spends waiting for weight stages (word 6) and for activation
            // slots (word 7), in ns
            unsigned long long wait_a = 0, wait_b = 0, tw;
#define LLMA_WAIT_BEGIN() (tw = globaltimer_ns())
#define LLMA_WAIT_END(acc) (acc += globaltimer_ns() - tw)
#else
#define LLMA_WAIT_BEGIN() ((void)0)
#define LLMA_WAIT_END(acc) ((void)0)
#endif
            for (int64_t w = w_beg; w < w_end && !sh[1]; ++seg) {
                const int tile = (int)(w / C), c0 = (int)(w - (int64_t)tile * C);
                const int c1 = (int)min((int64_t)C, c0 + (w_end - w));
                const int buf = n_acc == 2 ? (seg & 1) : 0;
                const uint32_t use = (uint32_t)(n_acc == 2 ? seg >> 1 : seg);
                if (!mbar_wait(acce_bar(buf), (use & 1u) ^ 1u)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * (uint32_t)acc_cols;
                for (int c = c0; c < c1 && !sh[1]; ++c, ++ia) {
                    LLMA_WAIT_BEGIN();
                    if (!mbar_wait(full_a(s), s_ph)) { atomicExch(g.dev_err, kDevErrTimeout); sh[1] = 1; break; }
                    LLMA_WAIT_END(wait_a);
                    if (ia == 0) LLMA_STAMP(stp, 2);
                    tc_fence_after();
                    const uint64_t da = smem_desc_sw128(sA + (uint32_t)s * stage_bytes);
                    const uint64_t db = smem_desc_sw128(sB + (uint32_t)s * stage_bytes);
                    const uint64_t db_lo = smem_desc_sw128(sB + (uint32_t)s * stage_bytes + (uint32_t)nr * 128u);
                    const uint32_t acc_on = c > c0 ? 1u : 0u;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {  // 4 x K=16 slices of the 64-wide chunk: +32 bytes each
                        umma_bf16(d_tmem, da + 2 * kk, db + 2 * kk, idesc, (acc_on || kk > 0) ? 1u : 0u);
                        if (!one_mma) umma_bf16(d_tmem + (uint32_t)nr, da + 2 * kk, db_lo + 2 * kk, idesc, (acc_on || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(empty_a(s));  // the stage is free once these MMAs have read it
                    if (++s == SA) { s = 0; s_ph ^= 1u; }
                }
                if (sh[1]) break;
                umma_commit(accf_bar(buf));  // accumulator complete
                LLMA_STAMP(stp, 3);
                w += c1 - c0;
            }
#ifdef LLMA_STAMPS
            if (stp) { stp[6] = wait_a; stp[7] = wait_b; }
#endif
        }
    } else {
        // ------------------------------- epilogue warps ------------------------------------------
        grid_dependency_wait();  // everything below reads or writes what earlier kernels produced
        if (threadIdx.x == 0) LLMA_STAMP(stp, 1);
        const int rows_used = g.rows ? min(g.rows->rows_used, g.nr) : g.nr;
        const int nr = wide_box_rows(g.nr, box_index(max(rows_used, 1)));  // as the MMA warp sees it
        const int acc_cols = 2 * nr;
        const int n_acc = 2 * acc_cols <= 512 ? 2 : 1;
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
        // stage up to 32 rows (jb .. jb + nj - 1, held in acc[0 .. nj - 1]) in shared memory, scaled by the folded
        // RMSNorm, then the fused epilogue
        auto finish_block = [&](int tile, int jb, int nj, float (&acc)[32]) {
            if (g.ss_in) {
#pragma unroll
                for (int j = 0; j < 32; ++j) stage[row][j] = acc[j] * rscale[min(jb + j, kRowCap - 1)];
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) stage[row][j] = acc[j];
            }
            epi_sync();
            if constexpr (MODE == kGemmQKV) {
                if (g.dims.head_dim == 128 || g.dims.head_dim == 64) epilogue_qkv_rows(g, tile, row, jb, nj, stage, s_pos, s_seq);
                else epilogue_qkv_wide(g, tile, row, jb, nj, stage, s_pos, s_seq);
            }
            else if constexpr (MODE == kGemmResid) {
                if ((g.n_out & 127) == 0) epilogue_resid_rows(g, tile, row, jb, nj, stage, red_f);
                else epilogue_resid<false>(g, tile, row, jb, nj, stage, red_f, xnone);
            } else if constexpr (MODE == kGemmSwiGLU) {
                if ((g.n_out & 15) == 0) epilogue_swiglu_rows(g, tile, row, jb, nj, stage);
                else epilogue_swiglu(g, tile, row, jb, nj, stage);
            }
            else if constexpr (MODE == kGemmStore) epilogue_store(g, tile, row, jb, nj, stage);
            else epilogue_lmhead(g, tile, row, jb, nj, stage, red_f, red_i);
            epi_sync();  // the staging area is rewritten by the next block
        };
        // Tiles cut by a range boundary are summed block by block: every CTA of such a tile writes its whole partial
        // (all-ones words while empty, see gemm_ws_kernel) into its own workspace slot -- slot 0 for the tile its
        // range begins in, slot 1 for any other -- and the tile's rows are dealt over its CTAs in blocks of 32 (of 16
        // where the tile has at least as many CTAs as 16-row blocks): after its last segment a CTA collects, for each
        // block dealt to it, the partials of all the tile's CTAs in ascending k order (its own among them), puts
        // all-ones back and runs the block's epilogue.  A tile cut into five
        // thus ends with five CTAs each finishing a fifth of it, instead of one CTA finishing all of it.
        constexpr uint32_t kEmpty = 0xFFFFFFFFu;
        // slots are laid out for the engine's row capacity whatever nr is: a prompt pass and a decoding step (different nr)
        // then agree on where every CTA's slots are
        const int qn = g.rc >> 2;
        const int tile_first = (int)(w_beg / C);
        bool aborted = false;
        int seg = 0;
        for (int64_t w = w_beg; w < w_end; ++seg) {
            const int tile = (int)(w / C), c0 = (int)(w - (int64_t)tile * C);
            const int c1 = (int)min((int64_t)C, c0 + (w_end - w));
            w += c1 - c0;
            const int buf = n_acc == 2 ? (seg & 1) : 0;
            const uint32_t use = (uint32_t)(n_acc == 2 ? seg >> 1 : seg);
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
            const int64_t t_lo = (int64_t)tile * C, t_hi = t_lo + C;
            const bool shared_tile = w_beg > t_lo || w_end < t_hi;
            const uint32_t t0 = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)buf * (uint32_t)acc_cols;
            for (int rb = 0; rb < nblk; ++rb) {
                float acc[32];
                tmem_ld_32cols(t0 + (uint32_t)rb * 32u, acc);
                {
                    float lo[32];
                    tmem_ld_32cols(t0 + (uint32_t)nr + (uint32_t)rb * 32u, lo);
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[j] += lo[j];  // W * hi + W * lo
                }
                if (shared_tile) {
                    float4* dst = ws_slot(g.ws, qn, b, tile == tile_first ? 0 : 1, row) + (int64_t)rb * 8 * 128;
#pragma unroll
                    for (int q = 0; q < 8; ++q)  // only the columns of rows in use travel
                        if (rb * 32 + 4 * q < rows_used) dst[q * 128] = make_float4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]);
                } else {
                    finish_block(tile, rb * 32, min(32, rows_used - rb * 32), acc);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(buf));  // MMA may overwrite this accumulator
        }
        if (!aborted && w_end > w_beg) {
            const unsigned long long give_up = globaltimer_ns() + 2000000000ull;
            bool timed_out = false;
            const int tile_last = (int)((w_end - 1) / C);
            for (int which = 0; which < 2; ++which) {
                const int tile = which == 0 ? tile_first : tile_last;
                if (which == 1 && tile_last == tile_first) break;
                const int64_t t_lo = (int64_t)tile * C, t_hi = t_lo + C;
                if (!(w_beg > t_lo || w_end < t_hi)) continue;  // the whole tile was this CTA's: finished above
                // the tile's CTAs: those whose ranges hold its first and its last chunk, and everyone between
                int b_first = (int)(t_lo * G / work);
                while (cta_begin(work, b_first + 1, G) <= t_lo) ++b_first;
                while (cta_begin(work, b_first, G) > t_lo) --b_first;
                int b_last = (int)((t_hi - 1) * G / work);
                while (cta_begin(work, b_last + 1, G) <= t_hi - 1) ++b_last;
                while (cta_begin(work, b_last, G) > t_hi - 1) --b_last;
                const int P = b_last - b_first + 1, me = b - b_first;
                // collect rows r_lo .. r_hi - 1 (NQ groups of four, starting at group q0 of 32-row block rb) from every
                // CTA of the tile in ascending k order, then run their epilogue; NQ is a compile-time 8 or 4 so that
                // the 32-row case carries no trace of the 16-row one
                auto collect = [&](auto nq_tag, int r_lo, int r_hi, int rb, int q0) {
                    constexpr int NQ = decltype(nq_tag)::value;
                    float acc[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[j] = 0.f;
                    for (int bb = b_first; bb <= b_last; ++bb) {  // ascending k: a fixed summation order
                        const int slot = (int)(cta_begin(work, bb, G) / C) == tile ? 0 : 1;
                        float4* src = ws_slot(g.ws, qn, bb, slot, row) + ((int64_t)rb * 8 + q0) * 128;
                        float4 p[NQ];
                        bool valid;
                        do {
                            valid = true;
#pragma unroll
                            for (int q = 0; q < NQ; ++q)
                                if (r_lo + 4 * q < r_hi) p[q] = ld_poll_f4(src + q * 128);
#pragma unroll
                            for (int q = 0; q < NQ; ++q) {
                                if (r_lo + 4 * q < r_hi) {
                                    valid = valid && __float_as_uint(p[q].x) != kEmpty;
                                    if (r_lo + 4 * q + 1 < r_hi) valid = valid && __float_as_uint(p[q].y) != kEmpty;
                                    if (r_lo + 4 * q + 2 < r_hi) valid = valid && __float_as_uint(p[q].z) != kEmpty;
                                    if (r_lo + 4 * q + 3 < r_hi) valid = valid && __float_as_uint(p[q].w) != kEmpty;
                                }
                            }
                            if (!valid && (timed_out || globaltimer_ns() > give_up)) {
                                atomicExch(g.dev_err, kDevErrTimeout); timed_out = true; break;
                            }
                        } while (!valid);
                        const float e = __uint_as_float(kEmpty);
#pragma unroll
                        for (int q = 0; q < NQ; ++q) {
                            if (r_lo + 4 * q < r_hi) {
                                src[q * 128] = make_float4(e, e, e, e);  // empty again for the next projection
                                acc[4 * q] += p[q].x; acc[4 * q + 1] += p[q].y; acc[4 * q + 2] += p[q].z; acc[4 * q + 3] += p[q].w;
                            }
                        }
                    }
                    finish_block(tile, r_lo, r_hi - r_lo, acc);
                };
                // units of 32 rows, or of 16 where that gives more of the tile's CTAs something to finish without
                // giving any of them two units
                if (nblk < P && ((rows_used + 15) >> 4) <= P) {
                    const int n_units = (rows_used + 15) >> 4;
                    for (int u = 0; u < n_units; ++u) {
                        if (u * P / n_units != me) continue;  // dealt to another CTA of the tile
                        const int r_lo = u * 16;
                        collect(std::integral_constant<int, 4>{}, r_lo, min(rows_used, r_lo + 16), r_lo >> 5, (r_lo & 31) >> 2);
                    }
                } else {
                    for (int rb = 0; rb < nblk; ++rb) {
                        if (rb * P / nblk != me) continue;
                        collect(std::integral_constant<int, 8>{}, rb * 32, min(rows_used, rb * 32 + 32), rb, 0);
                    }
                }
            }
        }
    }
    if (threadIdx.x == 0) LLMA_STAMP(stp, 5);
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
    c.b_slot = (uint32_t)nr * 256u;
    const size_t budget = (size_t)227 * 1024 - 1024 - kWideStageBytes - kWideTailBytes;
    const size_t stage_bytes = kGemmABytes + c.b_slot;
    // As many stages as fit, at most 8; an even number where there are four or more, because two lanes of each
    // producer warp take turns (a stage must always be refilled by the same lane: a lane that waited for "released
    // for the second time" on a stage whose first release it never waited for could be let through by the parity
    // of a barrier that has not completed any phase yet).  With two or three stages one lane issues.
    int S = (int)(budget / stage_bytes);
    if (S > 8) S = 8;
    if (S >= 4) S &= ~1;
    c.sa = c.sb = S;
    uint32_t cols = 32;
    for (int i = 0; i < 4; ++i) {  // the largest need over the row counts a step may choose (as in the kernel)
        const uint32_t acc_cols = 2u * (uint32_t)wide_box_rows(nr, i);
        while (cols < (2u * acc_cols <= 512u ? 2u : 1u) * acc_cols) cols <<= 1;
    }
    c.tmem_cols = cols;
    c.smem_bytes = 1024 + (size_t)S * stage_bytes + kWideStageBytes + kWideTailBytes;
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
                      const CUtensorMap& a1, const CUtensorMap& a2, const CUtensorMap* map_b) {
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
    const int sa = c.sa;
    const uint32_t cols = c.tmem_cols;
    switch (args.mode) {
        case kGemmQKV: cudaLaunchKernelEx(&cfg, gemm_wide_kernel<kGemmQKV>, args, a0, a1, a2, map_b[0], map_b[1], map_b[2], map_b[3], sa, cols); break;
        case kGemmResid: cudaLaunchKernelEx(&cfg, gemm_wide_kernel<kGemmResid>, args, a0, a1, a2, map_b[0], map_b[1], map_b[2], map_b[3], sa, cols); break;
        case kGemmSwiGLU: cudaLaunchKernelEx(&cfg, gemm_wide_kernel<kGemmSwiGLU>, args, a0, a1, a2, map_b[0], map_b[1], map_b[2], map_b[3], sa, cols); break;
        case kGemmLmHead: cudaLaunchKernelEx(&cfg, gemm_wide_kernel<kGemmLmHead>, args, a0, a1, a2, map_b[0], map_b[1], map_b[2], map_b[3], sa, cols); break;
        default: cudaLaunchKernelEx(&cfg, gemm_wide_kernel<kGemmStore>, args, a0, a1, a2, map_b[0], map_b[1], map_b[2], map_b[3], sa, cols); break;
    }
}

}  // namespace llma
