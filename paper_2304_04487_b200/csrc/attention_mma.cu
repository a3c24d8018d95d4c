// Split-KV causal attention for the k+1 query rows of a step (bf16 K/V cache).
//
// Grid (chunk, head, sequence).  A CTA owns 128 consecutive cache positions of one head:
// its K and V tiles arrive by TMA (128-byte swizzle) and are read ONCE for all the rows of
// the step, which is what makes verification of k+1 positions cost the K/V traffic of one.
// Each of the 4 warps takes 32 of the positions: S = Q K^T and O = P V on the tensor cores
// (mma.sync m16n8k16, bf16 in, fp32 accumulate), softmax statistics by warp shuffles.
// Q and P enter the MMAs as hi + lo bf16 pairs, so they keep 16 mantissa bits; Q is loaded
// from global memory directly into operand registers with all loads in flight at once, which
// keeps a CTA at 73 KB of shared memory: three CTAs per SM, one wave up to about 1.8 k cached
// positions at 32 heads.
#include <cuda.h>

#include "attention_mma.cuh"
#include "ptx_sm100.cuh"

namespace llma {

using namespace ptx;

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// (hi, lo) bf16 pairs of two floats, packed for an MMA operand register (x in the low half)
__device__ __forceinline__ void split_pack(float x, float y, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat16 xh = __float2bfloat16_rn(x), yh = __float2bfloat16_rn(y);
    const __nv_bfloat16 xl = __float2bfloat16_rn(x - __bfloat162float(xh));
    const __nv_bfloat16 yl = __float2bfloat16_rn(y - __bfloat162float(yh));
    hi = (uint32_t)__bfloat16_as_ushort(xh) | ((uint32_t)__bfloat16_as_ushort(yh) << 16);
    lo = (uint32_t)__bfloat16_as_ushort(xl) | ((uint32_t)__bfloat16_as_ushort(yl) << 16);
}

template <int HD>
struct AttnSmem {
    static constexpr int kBoxes = HD / 64;                    // 64-column TMA boxes per K (or V) tile
    static constexpr uint32_t kBoxBytes = kAttnChunk * 128;   // 128 rows x 128 bytes
    static constexpr uint32_t kTileBytes = kBoxes * kBoxBytes;
    static constexpr uint32_t offK = 0, offV = kTileBytes;
    static constexpr uint32_t offO = 2 * kTileBytes;                     // fp32 [16][HD] merged tile
    static constexpr uint32_t offStat = offO + 16 * HD * 4;              // m_w[4][16], l_w[4][16], misc
    static constexpr uint32_t kBytes = offStat + 2 * 4 * 16 * 4 + 64 + kRowCap * 4 + 16;  // + row positions, barriers
};

template <int HD, bool kPrompt>
__global__ void __launch_bounds__(128, 3) attention_mma_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap map_k,
                                                            const __grid_constant__ CUtensorMap map_v) {
    using L = AttnSmem<HD>;
    pdl_trigger();
    const int chunk = blockIdx.x, head = blockIdx.y, seq = blockIdx.z;
    // timeline (min, max over the CTAs): 0/1 CTA start, 2/3 dependency released, 4/5 K tile landed, 6/7 CTA end
    [[maybe_unused]] unsigned long long* stp = LLMA_STAMP_PTR(a.stamps, 300 + a.layer, 0);
    if (threadIdx.x == 0) LLMA_STAMP_MINMAX(stp, 0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const ModelDims& d = a.dims;
    const int c0 = chunk * kAttnChunk;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
    float* sO = reinterpret_cast<float*>(gbase + L::offO);
    float* s_m = reinterpret_cast<float*>(gbase + L::offStat);   // [4][16]
    float* s_l = s_m + 64;                                        // [4][16]
    uint64_t* bar = reinterpret_cast<uint64_t*>(s_l + 64);
    volatile uint32_t* flag = reinterpret_cast<volatile uint32_t*>(bar + 2);
    const uint32_t bar_u = smem_u32(bar), bar_v = bar_u + 8;  // K tile, V tile
    int* s_pos = reinterpret_cast<int*>(const_cast<uint32_t*>(flag) + 2);  // positions of this sequence's rows

    auto fetch_kv = [&]() {  // one thread
        const int32_t row0 = (int32_t)kv_row_index(d, a.layer, seq, head, c0);
        // K first, on a barrier of its own: S = Q K^T and the softmax run while V is still arriving
        mbar_arrive_expect_tx(bar_u, L::kTileBytes);
        for (int b = 0; b < L::kBoxes; ++b) tma_load_2d(base + L::offK + b * L::kBoxBytes, &map_k, bar_u, b * 64, row0);
        mbar_arrive_expect_tx(bar_v, L::kTileBytes);
        for (int b = 0; b < L::kBoxes; ++b) tma_load_2d(base + L::offV + b * L::kBoxBytes, &map_v, bar_v, b * 64, row0);
    };
    // A chunk that lies wholly below the length committed before this step cannot change during the step
    // (new K/V rows go to positions at or above that length), so its tiles are requested before waiting
    // for the QKV projection: the loads overlap that kernel's tail.
    const bool early = a.early_kv && c0 + kAttnChunk <= __ldcg(&a.seq_state[seq].kv_len);
    if (threadIdx.x == 0) {
        mbar_init(bar_u, 1); mbar_init(bar_v, 1); fence_mbar_init(); flag[0] = 0; flag[1] = 0;
        if (early) fetch_kv();
    }
    pdl_wait();  // row descriptors, q and the K/V rows of this step come from the kernels before
    if (threadIdx.x == 0) LLMA_STAMP_MINMAX(stp, 2);

    // rows of this sequence in the step (contiguous; summarised by the planning kernel)
    const int first = __ldcg(&a.rows->seq_first[seq]), cnt = __ldcg(&a.rows->seq_cnt[seq]);
    const int maxpos = __ldcg(&a.rows->seq_maxpos[seq]);
    if (cnt == 0 || c0 > maxpos) {  // uniform over the CTA; tiles already requested must land before the CTA goes
        if (early && threadIdx.x == 0) { (void)mbar_wait(bar_u, 0); (void)mbar_wait(bar_v, 0); }
        return;
    }
    for (int i = threadIdx.x; i < cnt; i += blockDim.x) s_pos[i] = __ldcg(&a.rows->pos[first + i]);
    __syncthreads();
    if (!early && threadIdx.x == 0) fetch_kv();
    // Q (this head, 16 of this sequence's rows) goes straight from global memory into the MMA's
    // A-operand registers as hi / lo bf16 pairs: lane (g, t) holds rows g and g + 8, columns
    // 16 ks + 2t, +1, +8, +9.  All loads are issued before any is used; rows past cnt are zero.
    const int g8 = lane >> 2, t4 = lane & 3;
    uint32_t qh[HD / 16][4], ql[HD / 16][4];
    auto load_q = [&](int mt) {
        const int r0 = mt * 16 + g8, r1 = r0 + 8;
        const int64_t ldq = 3 * (int64_t)d.hd_total;
        const float* q0 = a.qkv + (first + r0) * ldq + head * HD + 2 * t4;
        const float* q1 = q0 + 8 * ldq;
        float2 x[HD / 16][4];
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
            const float2 z = make_float2(0.f, 0.f);
            x[ks][0] = r0 < cnt ? __ldcg(reinterpret_cast<const float2*>(q0 + ks * 16)) : z;
            x[ks][1] = r1 < cnt ? __ldcg(reinterpret_cast<const float2*>(q1 + ks * 16)) : z;
            x[ks][2] = r0 < cnt ? __ldcg(reinterpret_cast<const float2*>(q0 + ks * 16 + 8)) : z;
            x[ks][3] = r1 < cnt ? __ldcg(reinterpret_cast<const float2*>(q1 + ks * 16 + 8)) : z;
        }
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
#pragma unroll
            for (int i = 0; i < 4; ++i) split_pack(x[ks][i].x, x[ks][i].y, qh[ks][i], ql[ks][i]);
        }
    };
    // The first tile's rows go through shared memory: the CTA fetches them as whole 16-byte accesses (a few per thread
    // instead of 32 eight-byte loads per lane, which filled the load/store queues once a sequence had more than a
    // row or two) into the buffer that later holds the merged tile, columns XOR-ed by (row & 3) * 8 so that the fragment
    // reads of a half-warp (four rows) fall into different banks.  With one or two rows the direct loads are few and
    // spare the barrier.
    if (cnt <= 2) {
        load_q(0);
    } else {
        float* sQ = sO;
        const int64_t ldq = 3 * (int64_t)d.hd_total;
        for (int idx = threadIdx.x; idx < 16 * (HD / 4); idx += blockDim.x) {
            const int r = idx / (HD / 4), c4 = idx - r * (HD / 4);
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < cnt) v = __ldcg(reinterpret_cast<const float4*>(a.qkv + (first + r) * ldq + head * HD) + c4);
            *reinterpret_cast<float4*>(sQ + r * HD + ((c4 * 4) ^ ((r & 3) << 3))) = v;
        }
        __syncthreads();
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = (i & 1) ? g8 + 8 : g8;
                const int col = ks * 16 + 2 * t4 + ((i >> 1) ? 8 : 0);
                const float2 x = *reinterpret_cast<const float2*>(sQ + row * HD + (col ^ ((row & 3) << 3)));
                split_pack(x.x, x.y, qh[ks][i], ql[ks][i]);
            }
        }
    }
    if (threadIdx.x == 0) {
        const bool ok = mbar_wait(bar_u, 0);
        if (!ok) { atomicExch(a.dev_err, kDevErrTimeout); flag[0] = 1; }
    }
    __syncthreads();
    if (flag[0]) return;  // the copy never landed: give up (error word is set)
    if (threadIdx.x == 0) LLMA_STAMP_MINMAX(stp, 4);

    const float scale = rsqrtf((float)HD);
    const int n_mt = (cnt + 15) >> 4;
    const int wpos0 = warp * 32;  // this warp's positions inside the chunk
    // chunk partials are indexed by the row's slot in the step: [head][chunk][row][HD]
    const int64_t part_base = ((int64_t)head * a.n_chunks + chunk) * d.row_cap + first;

    if (kPrompt && n_mt >= 4) {
        // Many rows of one sequence (prompt passes; an instance of its own, so that the decoding steps' instance keeps its registers): every warp takes whole 16-row query tiles (tile w, w + 4, ...) against
        // all 128 positions of the chunk, 32 positions at a time with a running maximum and sum, so that nothing is
        // combined across warps and no barrier separates the tiles.  A row's partial still depends on its position and
        // on the chunk only.
        const int mi = lane >> 3, t8 = lane & 7;
        bool v_ready = false;
        for (int mt = warp; mt < n_mt; mt += 4) {
            load_q(mt);
            const int r_lo = mt * 16 + g8, r_hi = r_lo + 8;
            const int lim_lo = r_lo < cnt ? s_pos[r_lo] : -1;
            const int lim_hi = r_hi < cnt ? s_pos[r_hi] : -1;
            const int lim_tile = s_pos[min(cnt - 1, mt * 16 + 15)];  // highest position of the tile (positions ascend with the row)
            float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
            float o[HD / 8][4];
#pragma unroll
            for (int i = 0; i < HD / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
#pragma unroll 1
            for (int sb = 0; sb < 4; ++sb) {
                const int wp0 = sb * 32;
                if (c0 + wp0 > lim_tile) break;  // warp-uniform: the rest of the chunk lies beyond every row of the tile
                float sc[4][4];
#pragma unroll
                for (int i = 0; i < 4; ++i) { sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f; }
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks) {
                    const uint32_t (&ah)[4] = qh[ks];
                    const uint32_t (&al)[4] = ql[ks];
#pragma unroll
                    for (int np = 0; np < 2; ++np) {
                        const int row = wp0 + np * 16 + (mi >> 1) * 8 + t8;
                        const int col = ks * 16 + (mi & 1) * 8;
                        const uint32_t kaddr = base + L::offK + (uint32_t)(col >> 6) * L::kBoxBytes + (uint32_t)row * 128 +
                                               ((((uint32_t)(col & 63) >> 3) ^ ((uint32_t)row & 7u)) << 4);
                        uint32_t b[4];
                        ldsm_x4(kaddr, b);
                        mma_bf16(sc[2 * np], ah, b[0], b[1]);
                        mma_bf16(sc[2 * np], al, b[0], b[1]);
                        mma_bf16(sc[2 * np + 1], ah, b[2], b[3]);
                        mma_bf16(sc[2 * np + 1], al, b[2], b[3]);
                    }
                }
                float bm_lo = -INFINITY, bm_hi = -INFINITY;
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int p = c0 + wp0 + nt * 8 + 2 * (lane & 3) + (e & 1);
                        const int lim = e < 2 ? lim_lo : lim_hi;
                        const float v = p <= lim ? sc[nt][e] * scale : -INFINITY;
                        sc[nt][e] = v;
                        if (e < 2) bm_lo = fmaxf(bm_lo, v); else bm_hi = fmaxf(bm_hi, v);
                    }
                }
                bm_lo = fmaxf(bm_lo, __shfl_xor_sync(0xffffffffu, bm_lo, 1)); bm_lo = fmaxf(bm_lo, __shfl_xor_sync(0xffffffffu, bm_lo, 2));
                bm_hi = fmaxf(bm_hi, __shfl_xor_sync(0xffffffffu, bm_hi, 1)); bm_hi = fmaxf(bm_hi, __shfl_xor_sync(0xffffffffu, bm_hi, 2));
                const float n_lo = fmaxf(m_lo, bm_lo), n_hi = fmaxf(m_hi, bm_hi);
                const float ref_lo = n_lo == -INFINITY ? 0.f : n_lo, ref_hi = n_hi == -INFINITY ? 0.f : n_hi;
                const float f_lo = m_lo == -INFINITY ? 0.f : expf(m_lo - ref_lo);  // what was gathered so far, on the new scale
                const float f_hi = m_hi == -INFINITY ? 0.f : expf(m_hi - ref_hi);
                float bl_lo = 0.f, bl_hi = 0.f;
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float pe = expf(sc[nt][e] - (e < 2 ? ref_lo : ref_hi));  // exp(-inf) = 0 for masked positions
                        sc[nt][e] = pe;
                        if (e < 2) bl_lo += pe; else bl_hi += pe;
                    }
                }
                bl_lo += __shfl_xor_sync(0xffffffffu, bl_lo, 1); bl_lo += __shfl_xor_sync(0xffffffffu, bl_lo, 2);
                bl_hi += __shfl_xor_sync(0xffffffffu, bl_hi, 1); bl_hi += __shfl_xor_sync(0xffffffffu, bl_hi, 2);
                l_lo = __fmaf_rn(l_lo, f_lo, bl_lo); l_hi = __fmaf_rn(l_hi, f_hi, bl_hi);
                m_lo = n_lo; m_hi = n_hi;
#pragma unroll
                for (int i = 0; i < HD / 8; ++i) { o[i][0] *= f_lo; o[i][1] *= f_lo; o[i][2] *= f_hi; o[i][3] *= f_hi; }
                if (!v_ready) {  // the V tile, once per warp
                    bool ok = true;
                    if (lane == 0) ok = mbar_wait(bar_v, 0);
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { if (lane == 0) atomicExch(a.dev_err, kDevErrTimeout); return; }
                    v_ready = true;
                }
#pragma unroll
                for (int kp = 0; kp < 2; ++kp) {
                    uint32_t ph[4], pl[4];
                    split_pack(sc[2 * kp][0], sc[2 * kp][1], ph[0], pl[0]);
                    split_pack(sc[2 * kp][2], sc[2 * kp][3], ph[1], pl[1]);
                    split_pack(sc[2 * kp + 1][0], sc[2 * kp + 1][1], ph[2], pl[2]);
                    split_pack(sc[2 * kp + 1][2], sc[2 * kp + 1][3], ph[3], pl[3]);
#pragma unroll
                    for (int nn = 0; nn < HD / 16; ++nn) {
                        const int row = wp0 + kp * 16 + (mi & 1) * 8 + t8;
                        const int col = nn * 16 + (mi >> 1) * 8;
                        const uint32_t vaddr = base + L::offV + (uint32_t)(col >> 6) * L::kBoxBytes + (uint32_t)row * 128 +
                                               ((((uint32_t)(col & 63) >> 3) ^ ((uint32_t)row & 7u)) << 4);
                        uint32_t b[4];
                        ldsm_x4_trans(vaddr, b);
                        mma_bf16(o[2 * nn], ph, b[0], b[1]);
                        mma_bf16(o[2 * nn], pl, b[0], b[1]);
                        mma_bf16(o[2 * nn + 1], ph, b[2], b[3]);
                        mma_bf16(o[2 * nn + 1], pl, b[2], b[3]);
                    }
                }
            }
            // the tile's partial of this chunk, straight from the fragments (rows past cnt are not written)
#pragma unroll
            for (int nt = 0; nt < HD / 8; ++nt) {
                const int col = nt * 8 + 2 * t4;
                if (r_lo < cnt) *reinterpret_cast<float2*>(a.ws_o + (part_base + r_lo) * HD + col) = make_float2(o[nt][0], o[nt][1]);
                if (r_hi < cnt) *reinterpret_cast<float2*>(a.ws_o + (part_base + r_hi) * HD + col) = make_float2(o[nt][2], o[nt][3]);
            }
            if (t4 == 0) {
                if (r_lo < cnt) { a.ws_ml[(part_base + r_lo) * 2] = m_lo; a.ws_ml[(part_base + r_lo) * 2 + 1] = l_lo; }
                if (r_hi < cnt) { a.ws_ml[(part_base + r_hi) * 2] = m_hi; a.ws_ml[(part_base + r_hi) * 2 + 1] = l_hi; }
            }
        }
        if (!v_ready && lane == 0) (void)mbar_wait(bar_v, 0);  // a copy in flight must land before the CTA's memory goes away
        if (threadIdx.x == 0) LLMA_STAMP_MINMAX(stp, 6);
        return;
    }
    for (int mt = 0; mt < n_mt; ++mt) {
        if (mt > 0) load_q(mt);
        // ---------------- S = Q K^T over this warp's 32 positions ----------------------------
        float s[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
        const int mi = lane >> 3, t8 = lane & 7;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
            const uint32_t (&ah)[4] = qh[ks];
            const uint32_t (&al)[4] = ql[ks];
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                const int row = wpos0 + np * 16 + (mi >> 1) * 8 + t8;
                const int col = ks * 16 + (mi & 1) * 8;
                const uint32_t kaddr = base + L::offK + (uint32_t)(col >> 6) * L::kBoxBytes + (uint32_t)row * 128 +
                                       ((((uint32_t)(col & 63) >> 3) ^ ((uint32_t)row & 7u)) << 4);
                uint32_t b[4];
                ldsm_x4(kaddr, b);
                mma_bf16(s[2 * np], ah, b[0], b[1]);
                mma_bf16(s[2 * np], al, b[0], b[1]);
                mma_bf16(s[2 * np + 1], ah, b[2], b[3]);
                mma_bf16(s[2 * np + 1], al, b[2], b[3]);
            }
        }
        // ---------------- causal mask, softmax statistics of the warp's span --------------------
        const int r_lo = mt * 16 + (lane >> 2), r_hi = r_lo + 8;
        const int lim_lo = r_lo < cnt ? s_pos[r_lo] : -1;
        const int lim_hi = r_hi < cnt ? s_pos[r_hi] : -1;
        float m_lo = -INFINITY, m_hi = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int p = c0 + wpos0 + nt * 8 + 2 * (lane & 3) + (e & 1);
                const int lim = e < 2 ? lim_lo : lim_hi;
                const float v = p <= lim ? s[nt][e] * scale : -INFINITY;
                s[nt][e] = v;
                if (e < 2) m_lo = fmaxf(m_lo, v); else m_hi = fmaxf(m_hi, v);
            }
        }
        m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 1)); m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 2));
        m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 1)); m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 2));
        const float ref_lo = m_lo == -INFINITY ? 0.f : m_lo, ref_hi = m_hi == -INFINITY ? 0.f : m_hi;
        float l_lo = 0.f, l_hi = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float pe = expf(s[nt][e] - (e < 2 ? ref_lo : ref_hi));  // exp(-inf) = 0 for masked positions
                s[nt][e] = pe;
                if (e < 2) l_lo += pe; else l_hi += pe;
            }
        }
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

        // ---------------- O = P V ----------------------------------------------------------------
        if (mt == 0) {
            if (threadIdx.x == 0 && !mbar_wait(bar_v, 0)) { atomicExch(a.dev_err, kDevErrTimeout); flag[0] = 1; }
            __syncthreads();
            if (flag[0]) return;  // uniform: the copy never landed (error word is set)
        }
        float o[HD / 8][4];
#pragma unroll
        for (int i = 0; i < HD / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
#pragma unroll
        for (int kp = 0; kp < 2; ++kp) {
            uint32_t ph[4], pl[4];
            split_pack(s[2 * kp][0], s[2 * kp][1], ph[0], pl[0]);
            split_pack(s[2 * kp][2], s[2 * kp][3], ph[1], pl[1]);
            split_pack(s[2 * kp + 1][0], s[2 * kp + 1][1], ph[2], pl[2]);
            split_pack(s[2 * kp + 1][2], s[2 * kp + 1][3], ph[3], pl[3]);
#pragma unroll
            for (int nn = 0; nn < HD / 16; ++nn) {
                const int row = wpos0 + kp * 16 + (mi & 1) * 8 + t8;
                const int col = nn * 16 + (mi >> 1) * 8;
                const uint32_t vaddr = base + L::offV + (uint32_t)(col >> 6) * L::kBoxBytes + (uint32_t)row * 128 +
                                       ((((uint32_t)(col & 63) >> 3) ^ ((uint32_t)row & 7u)) << 4);
                uint32_t b[4];
                ldsm_x4_trans(vaddr, b);
                mma_bf16(o[2 * nn], ph, b[0], b[1]);
                mma_bf16(o[2 * nn], pl, b[0], b[1]);
                mma_bf16(o[2 * nn + 1], ph, b[2], b[3]);
                mma_bf16(o[2 * nn + 1], pl, b[2], b[3]);
            }
        }
        // ---------------- merge the 4 warps in warp order, chunk partial -> workspace -----------------
        if ((lane & 3) == 0) {
            s_m[warp * 16 + (lane >> 2)] = m_lo; s_m[warp * 16 + (lane >> 2) + 8] = m_hi;
            s_l[warp * 16 + (lane >> 2)] = l_lo; s_l[warp * 16 + (lane >> 2) + 8] = l_hi;
        }
        const int rows_here = min(16, cnt - mt * 16);
        if (n_mt == 1) {
            // The K tile is dead (every warp passed the barrier after its scores): each warp parks its
            // unscaled partial there, [warp][16 rows][HD] with the column XOR-ed by (row & 3) * 8 so that
            // neither the stores nor the float4 reads below conflict; then all threads combine the four
            // partials of their elements in warp order and write the chunk's partial straight to global memory.
            float* buf = reinterpret_cast<float*>(gbase + L::offK) + warp * 16 * HD;
#pragma unroll
            for (int nt = 0; nt < HD / 8; ++nt) {
                const int col = nt * 8 + 2 * t4;
                *reinterpret_cast<float2*>(buf + g8 * HD + (col ^ ((g8 & 3) << 3))) = make_float2(o[nt][0], o[nt][1]);
                *reinterpret_cast<float2*>(buf + (g8 + 8) * HD + (col ^ ((g8 & 3) << 3))) = make_float2(o[nt][2], o[nt][3]);
            }
            __syncthreads();
            const float* all = reinterpret_cast<const float*>(gbase + L::offK);
            for (int e = threadIdx.x; e < rows_here * (HD / 4); e += blockDim.x) {
                const int r = e / (HD / 4), c4 = e - r * (HD / 4);
                float M = -INFINITY;
#pragma unroll
                for (int w = 0; w < 4; ++w) M = fmaxf(M, s_m[w * 16 + r]);
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const float mw = s_m[w * 16 + r];
                    const float f = mw == -INFINITY ? 0.f : expf(mw - M);
                    const float4 v = *reinterpret_cast<const float4*>(all + (w * 16 + r) * HD + ((c4 * 4) ^ ((r & 3) << 3)));
                    if (w == 0) {
                        acc = make_float4(__fmul_rn(f, v.x), __fmul_rn(f, v.y), __fmul_rn(f, v.z), __fmul_rn(f, v.w));
                    } else {
                        acc.x = __fmaf_rn(f, v.x, acc.x); acc.y = __fmaf_rn(f, v.y, acc.y);
                        acc.z = __fmaf_rn(f, v.z, acc.z); acc.w = __fmaf_rn(f, v.w, acc.w);
                    }
                }
                *reinterpret_cast<float4*>(a.ws_o + (part_base + r) * HD + c4 * 4) = acc;
            }
        } else {
            // several 16-row tiles share the K and V tiles: accumulate in a buffer of its own, warp by warp
            // (the same products and fused multiply-adds as above, so a row's bits do not depend on the path)
            __syncthreads();
            float M_lo = -INFINITY, M_hi = -INFINITY;
#pragma unroll
            for (int w = 0; w < 4; ++w) { M_lo = fmaxf(M_lo, s_m[w * 16 + (lane >> 2)]); M_hi = fmaxf(M_hi, s_m[w * 16 + (lane >> 2) + 8]); }
            const float f_lo = m_lo == -INFINITY ? 0.f : expf(m_lo - M_lo);
            const float f_hi = m_hi == -INFINITY ? 0.f : expf(m_hi - M_hi);
            for (int w = 0; w < 4; ++w) {
                if (warp == w) {
#pragma unroll
                    for (int nt = 0; nt < HD / 8; ++nt) {
                        float* p_lo = sO + (lane >> 2) * HD + nt * 8 + 2 * (lane & 3);
                        float* p_hi = p_lo + 8 * HD;
                        if (w == 0) {
                            p_lo[0] = __fmul_rn(f_lo, o[nt][0]); p_lo[1] = __fmul_rn(f_lo, o[nt][1]);
                            p_hi[0] = __fmul_rn(f_hi, o[nt][2]); p_hi[1] = __fmul_rn(f_hi, o[nt][3]);
                        } else {
                            p_lo[0] = __fmaf_rn(f_lo, o[nt][0], p_lo[0]); p_lo[1] = __fmaf_rn(f_lo, o[nt][1], p_lo[1]);
                            p_hi[0] = __fmaf_rn(f_hi, o[nt][2], p_hi[0]); p_hi[1] = __fmaf_rn(f_hi, o[nt][3], p_hi[1]);
                        }
                    }
                }
                __syncthreads();
            }
            for (int idx = threadIdx.x; idx < rows_here * HD; idx += blockDim.x) {
                const int r = idx / HD, i = idx - r * HD;
                a.ws_o[(part_base + mt * 16 + r) * HD + i] = sO[r * HD + i];
            }
        }
        if (threadIdx.x < rows_here) {
            const int r = threadIdx.x;
            float M = -INFINITY;
            for (int w = 0; w < 4; ++w) M = fmaxf(M, s_m[w * 16 + r]);
            float lsum = 0.f;
            for (int w = 0; w < 4; ++w) {
                const float mw = s_m[w * 16 + r];
                lsum += mw == -INFINITY ? 0.f : expf(mw - M) * s_l[w * 16 + r];
            }
            a.ws_ml[(part_base + mt * 16 + r) * 2] = M;
            a.ws_ml[(part_base + mt * 16 + r) * 2 + 1] = lsum;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) LLMA_STAMP_MINMAX(stp, 6);
}

// Long contexts, many sequences: a CTA takes kT consecutive 128-position tiles of one (sequence, head) instead of one,
// so that the chunk partials (and the merge pass over them) shrink by kT and the next tile's K and V are already on
// their way while the current one is being multiplied.  Each warp keeps its 32-position slice's running maximum, sum
// and output across the tiles; the four warps are combined once, at the end, exactly as in attention_mma_kernel.
// For steps of at most 16 rows per sequence; which kT an engine uses depends on its capacity only (never on the step).
template <int HD, int kT>
__global__ void __launch_bounds__(128, 3) attention_long_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap map_k,
                                                             const __grid_constant__ CUtensorMap map_v) {
    using L = AttnSmem<HD>;
    pdl_trigger();
    const int chunk = blockIdx.x, head = blockIdx.y, seq = blockIdx.z;
    [[maybe_unused]] unsigned long long* stp = LLMA_STAMP_PTR(a.stamps, 300 + a.layer, 0);
    if (threadIdx.x == 0) LLMA_STAMP_MINMAX(stp, 0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const ModelDims& d = a.dims;
    const int c0 = chunk * kAttnChunk * kT;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
    float* sO = reinterpret_cast<float*>(gbase + L::offO);
    float* s_m = reinterpret_cast<float*>(gbase + L::offStat);   // [4][16]
    float* s_l = s_m + 64;                                        // [4][16]
    uint64_t* bar = reinterpret_cast<uint64_t*>(s_l + 64);
    volatile uint32_t* flag = reinterpret_cast<volatile uint32_t*>(bar + 2);
    const uint32_t bar_u = smem_u32(bar), bar_v = bar_u + 8;  // K tile, V tile
    int* s_pos = reinterpret_cast<int*>(const_cast<uint32_t*>(flag) + 2);

    auto fetch_k = [&](int t) {  // one thread
        const int32_t row0 = (int32_t)kv_row_index(d, a.layer, seq, head, c0 + t * kAttnChunk);
        mbar_arrive_expect_tx(bar_u, L::kTileBytes);
        for (int b = 0; b < L::kBoxes; ++b) tma_load_2d(base + L::offK + b * L::kBoxBytes, &map_k, bar_u, b * 64, row0);
    };
    auto fetch_v = [&](int t) {
        const int32_t row0 = (int32_t)kv_row_index(d, a.layer, seq, head, c0 + t * kAttnChunk);
        mbar_arrive_expect_tx(bar_v, L::kTileBytes);
        for (int b = 0; b < L::kBoxes; ++b) tma_load_2d(base + L::offV + b * L::kBoxBytes, &map_v, bar_v, b * 64, row0);
    };
    // the first tile may be requested before the QKV projection has finished if it lies wholly below the committed length
    const bool early = a.early_kv && c0 + kAttnChunk <= __ldcg(&a.seq_state[seq].kv_len);
    if (threadIdx.x == 0) {
        mbar_init(bar_u, 1); mbar_init(bar_v, 1); fence_mbar_init(); flag[0] = 0; flag[1] = 0;
        if (early) { fetch_k(0); fetch_v(0); }
    }
    pdl_wait();
    if (threadIdx.x == 0) LLMA_STAMP_MINMAX(stp, 2);

    const int first = __ldcg(&a.rows->seq_first[seq]), cnt = __ldcg(&a.rows->seq_cnt[seq]);
    const int maxpos = __ldcg(&a.rows->seq_maxpos[seq]);
    if (cnt == 0 || c0 > maxpos) {
        if (early && threadIdx.x == 0) { (void)mbar_wait(bar_u, 0); (void)mbar_wait(bar_v, 0); }
        return;
    }
    if (cnt > 16) {  // not this kernel's case: the host never launches it for such steps
        if (threadIdx.x == 0) {
            atomicExch(a.dev_err, kDevErrCapacity);
            if (early) { (void)mbar_wait(bar_u, 0); (void)mbar_wait(bar_v, 0); }
        }
        return;
    }
    for (int i = threadIdx.x; i < cnt; i += blockDim.x) s_pos[i] = __ldcg(&a.rows->pos[first + i]);
    __syncthreads();
    if (!early && threadIdx.x == 0) { fetch_k(0); fetch_v(0); }
    const int n_tiles = min(kT, (maxpos - c0) / kAttnChunk + 1);  // tiles that hold a position some row attends to

    const int g8 = lane >> 2, t4 = lane & 3;
    uint32_t qh[HD / 16][4], ql[HD / 16][4];
    {   // the step's rows of q for this head through shared memory (see attention_mma_kernel)
        float* sQ = sO;
        const int64_t ldq = 3 * (int64_t)d.hd_total;
        for (int idx = threadIdx.x; idx < 16 * (HD / 4); idx += blockDim.x) {
            const int r = idx / (HD / 4), c4 = idx - r * (HD / 4);
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < cnt) v = __ldcg(reinterpret_cast<const float4*>(a.qkv + (first + r) * ldq + head * HD) + c4);
            *reinterpret_cast<float4*>(sQ + r * HD + ((c4 * 4) ^ ((r & 3) << 3))) = v;
        }
        __syncthreads();
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = (i & 1) ? g8 + 8 : g8;
                const int col = ks * 16 + 2 * t4 + ((i >> 1) ? 8 : 0);
                const float2 x = *reinterpret_cast<const float2*>(sQ + row * HD + (col ^ ((row & 3) << 3)));
                split_pack(x.x, x.y, qh[ks][i], ql[ks][i]);
            }
        }
    }
    const float scale = rsqrtf((float)HD);
    const int wpos0 = warp * 32;
    const int mi = lane >> 3, t8 = lane & 7;
    const int r_lo = g8, r_hi = g8 + 8;
    const int lim_lo = r_lo < cnt ? s_pos[r_lo] : -1;
    const int lim_hi = r_hi < cnt ? s_pos[r_hi] : -1;
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
    float o[HD / 8][4];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }

#pragma unroll 1
    for (int t = 0; t < n_tiles; ++t) {
        const uint32_t par = (uint32_t)(t & 1);
        if (threadIdx.x == 0 && !mbar_wait(bar_u, par)) { atomicExch(a.dev_err, kDevErrTimeout); flag[0] = 1; }
        __syncthreads();
        if (flag[0]) break;  // uniform; what is still in flight is awaited below
        if (t == 0 && threadIdx.x == 0) LLMA_STAMP_MINMAX(stp, 4);
        float sc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
            const uint32_t (&ah)[4] = qh[ks];
            const uint32_t (&al)[4] = ql[ks];
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                const int row = wpos0 + np * 16 + (mi >> 1) * 8 + t8;
                const int col = ks * 16 + (mi & 1) * 8;
                const uint32_t kaddr = base + L::offK + (uint32_t)(col >> 6) * L::kBoxBytes + (uint32_t)row * 128 +
                                       ((((uint32_t)(col & 63) >> 3) ^ ((uint32_t)row & 7u)) << 4);
                uint32_t b[4];
                ldsm_x4(kaddr, b);
                mma_bf16(sc[2 * np], ah, b[0], b[1]);
                mma_bf16(sc[2 * np], al, b[0], b[1]);
                mma_bf16(sc[2 * np + 1], ah, b[2], b[3]);
                mma_bf16(sc[2 * np + 1], al, b[2], b[3]);
            }
        }
        __syncthreads();  // every warp has read the K tile: the next one may land in it
        if (threadIdx.x == 0 && t + 1 < n_tiles) fetch_k(t + 1);
        const int p0 = c0 + t * kAttnChunk + wpos0;
        float bm_lo = -INFINITY, bm_hi = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int p = p0 + nt * 8 + 2 * (lane & 3) + (e & 1);
                const int lim = e < 2 ? lim_lo : lim_hi;
                const float v = p <= lim ? sc[nt][e] * scale : -INFINITY;
                sc[nt][e] = v;
                if (e < 2) bm_lo = fmaxf(bm_lo, v); else bm_hi = fmaxf(bm_hi, v);
            }
        }
        bm_lo = fmaxf(bm_lo, __shfl_xor_sync(0xffffffffu, bm_lo, 1)); bm_lo = fmaxf(bm_lo, __shfl_xor_sync(0xffffffffu, bm_lo, 2));
        bm_hi = fmaxf(bm_hi, __shfl_xor_sync(0xffffffffu, bm_hi, 1)); bm_hi = fmaxf(bm_hi, __shfl_xor_sync(0xffffffffu, bm_hi, 2));
        const float n_lo = fmaxf(m_lo, bm_lo), n_hi = fmaxf(m_hi, bm_hi);
        const float ref_lo = n_lo == -INFINITY ? 0.f : n_lo, ref_hi = n_hi == -INFINITY ? 0.f : n_hi;
        const float f_lo = m_lo == -INFINITY ? 0.f : expf(m_lo - ref_lo);
        const float f_hi = m_hi == -INFINITY ? 0.f : expf(m_hi - ref_hi);
        float bl_lo = 0.f, bl_hi = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float pe = expf(sc[nt][e] - (e < 2 ? ref_lo : ref_hi));
                sc[nt][e] = pe;
                if (e < 2) bl_lo += pe; else bl_hi += pe;
            }
        }
        bl_lo += __shfl_xor_sync(0xffffffffu, bl_lo, 1); bl_lo += __shfl_xor_sync(0xffffffffu, bl_lo, 2);
        bl_hi += __shfl_xor_sync(0xffffffffu, bl_hi, 1); bl_hi += __shfl_xor_sync(0xffffffffu, bl_hi, 2);
        l_lo = __fmaf_rn(l_lo, f_lo, bl_lo); l_hi = __fmaf_rn(l_hi, f_hi, bl_hi);
        m_lo = n_lo; m_hi = n_hi;
#pragma unroll
        for (int i = 0; i < HD / 8; ++i) { o[i][0] *= f_lo; o[i][1] *= f_lo; o[i][2] *= f_hi; o[i][3] *= f_hi; }
        if (threadIdx.x == 0 && !mbar_wait(bar_v, par)) { atomicExch(a.dev_err, kDevErrTimeout); flag[0] = 1; }
        __syncthreads();
        if (flag[0]) break;
#pragma unroll
        for (int kp = 0; kp < 2; ++kp) {
            uint32_t ph[4], pl[4];
            split_pack(sc[2 * kp][0], sc[2 * kp][1], ph[0], pl[0]);
            split_pack(sc[2 * kp][2], sc[2 * kp][3], ph[1], pl[1]);
            split_pack(sc[2 * kp + 1][0], sc[2 * kp + 1][1], ph[2], pl[2]);
            split_pack(sc[2 * kp + 1][2], sc[2 * kp + 1][3], ph[3], pl[3]);
#pragma unroll
            for (int nn = 0; nn < HD / 16; ++nn) {
                const int row = wpos0 + kp * 16 + (mi & 1) * 8 + t8;
                const int col = nn * 16 + (mi >> 1) * 8;
                const uint32_t vaddr = base + L::offV + (uint32_t)(col >> 6) * L::kBoxBytes + (uint32_t)row * 128 +
                                       ((((uint32_t)(col & 63) >> 3) ^ ((uint32_t)row & 7u)) << 4);
                uint32_t b[4];
                ldsm_x4_trans(vaddr, b);
                mma_bf16(o[2 * nn], ph, b[0], b[1]);
                mma_bf16(o[2 * nn], pl, b[0], b[1]);
                mma_bf16(o[2 * nn + 1], ph, b[2], b[3]);
                mma_bf16(o[2 * nn + 1], pl, b[2], b[3]);
            }
        }
        __syncthreads();  // every warp has read the V tile
        if (threadIdx.x == 0 && t + 1 < n_tiles) fetch_v(t + 1);
    }
    if (flag[0]) {
        // a copy never landed (error word is set): the K copy of the next tile may still be in flight
        if (threadIdx.x == 0) {
            (void)mbar_wait(bar_u, 0, 100000000ull); (void)mbar_wait(bar_u, 1, 100000000ull);
            (void)mbar_wait(bar_v, 0, 100000000ull); (void)mbar_wait(bar_v, 1, 100000000ull);
        }
        return;
    }
    // ---------------- the four warps' (max, sum, output) combined in warp order -> the chunk's partial ----------------
    const int64_t part_base = ((int64_t)head * a.n_chunks + chunk) * d.row_cap + first;
    if ((lane & 3) == 0) {
        s_m[warp * 16 + g8] = m_lo; s_m[warp * 16 + g8 + 8] = m_hi;
        s_l[warp * 16 + g8] = l_lo; s_l[warp * 16 + g8 + 8] = l_hi;
    }
    {
        float* buf = reinterpret_cast<float*>(gbase + L::offK) + warp * 16 * HD;  // the K tile is dead
#pragma unroll
        for (int nt = 0; nt < HD / 8; ++nt) {
            const int col = nt * 8 + 2 * t4;
            *reinterpret_cast<float2*>(buf + g8 * HD + (col ^ ((g8 & 3) << 3))) = make_float2(o[nt][0], o[nt][1]);
            *reinterpret_cast<float2*>(buf + (g8 + 8) * HD + (col ^ ((g8 & 3) << 3))) = make_float2(o[nt][2], o[nt][3]);
        }
        __syncthreads();
        const float* all = reinterpret_cast<const float*>(gbase + L::offK);
        for (int e = threadIdx.x; e < cnt * (HD / 4); e += blockDim.x) {
            const int r = e / (HD / 4), c4 = e - r * (HD / 4);
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < 4; ++w) M = fmaxf(M, s_m[w * 16 + r]);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const float mw = s_m[w * 16 + r];
                const float f = mw == -INFINITY ? 0.f : expf(mw - M);
                const float4 v = *reinterpret_cast<const float4*>(all + (w * 16 + r) * HD + ((c4 * 4) ^ ((r & 3) << 3)));
                if (w == 0) {
                    acc = make_float4(__fmul_rn(f, v.x), __fmul_rn(f, v.y), __fmul_rn(f, v.z), __fmul_rn(f, v.w));
                } else {
                    acc.x = __fmaf_rn(f, v.x, acc.x); acc.y = __fmaf_rn(f, v.y, acc.y);
                    acc.z = __fmaf_rn(f, v.z, acc.z); acc.w = __fmaf_rn(f, v.w, acc.w);
                }
            }
            *reinterpret_cast<float4*>(a.ws_o + (part_base + r) * HD + c4 * 4) = acc;
        }
    }
    if (threadIdx.x < cnt) {
        const int r = threadIdx.x;
        float M = -INFINITY;
        for (int w = 0; w < 4; ++w) M = fmaxf(M, s_m[w * 16 + r]);
        float lsum = 0.f;
        for (int w = 0; w < 4; ++w) {
            const float mw = s_m[w * 16 + r];
            lsum += mw == -INFINITY ? 0.f : expf(mw - M) * s_l[w * 16 + r];
        }
        a.ws_ml[(part_base + r) * 2] = M;
        a.ws_ml[(part_base + r) * 2 + 1] = lsum;
    }
    if (threadIdx.x == 0) LLMA_STAMP_MINMAX(stp, 6);
}

// Second pass: one warp per (head, row) combines the row's chunk partials in ascending chunk
// order.  A kernel of its own, so that every head is merged at once instead of by whichever CTA of the
// head happened to finish last; a row's result still depends on its own position only.
template <int HD>
__global__ void __launch_bounds__(128) attention_merge_kernel(const AttnArgs a) {
    pdl_trigger();
    // timeline (min, max over the warps): 2/3 dependency released, 6/7 warp end
    [[maybe_unused]] unsigned long long* stp = LLMA_STAMP_PTR(a.stamps, 400 + a.layer, 0);
    pdl_wait();
    if ((threadIdx.x & 31) == 0) LLMA_STAMP_MINMAX(stp, 2);
    extern __shared__ float s_w[];  // [4 warps][n_chunks] weights, then [4][n_chunks] weighted sums
    const int head = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const ModelDims& d = a.dims;
    const int r = blockIdx.y * 4 + warp;  // row slot of the step (below the pass's row slots: they come in fours)
    const int64_t head_base = (int64_t)head * a.n_chunks * d.row_cap;
    float* w_c = s_w + warp * a.n_chunks;
    float* wl_c = s_w + (4 + warp) * a.n_chunks;
    // The kernel is a chain of dependent loads, so everything whose address is known is requested at once:
    // the row's position, the (max, sum) pairs of every chunk slot and the first sixteen chunk partials.
    // Slots past the row's last chunk hold older (finite) values; they are read but never used.
    const int rows_used = __ldcg(&a.rows->rows_used);
    const int pos = __ldcg(&a.rows->pos[r]);
    // a step shaped for many rows (batched decoding) usually uses a fraction of its row slots: there a warp first
    // learns whether its slot is in use, at the price of one more round trip for those that are
    if (a.n_rows > 32 && (r >= rows_used || pos < 0)) return;
    const float4* src = reinterpret_cast<const float4*>(a.ws_o + (head_base + r) * HD) + (lane < HD / 4 ? lane : 0);
    float2 ml[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int c = lane + 32 * u;
        ml[u] = c < a.n_chunks ? __ldcg(reinterpret_cast<const float2*>(a.ws_ml) + head_base + (int64_t)c * d.row_cap + r)
                               : make_float2(-INFINITY, 0.f);
    }
    float4 p0[16];
#pragma unroll
    for (int u = 0; u < 16; ++u)
        p0[u] = u < a.n_chunks ? __ldcg(src + (int64_t)u * d.row_cap * (HD / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
    if (r >= rows_used || pos < 0) return;
    const int nc = pos / a.chunk_pos + 1;
    float M = -INFINITY;
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int c = lane + 32 * u;
        if (c < nc) { w_c[c] = ml[u].x; wl_c[c] = ml[u].y; M = fmaxf(M, ml[u].x); }
    }
    for (int c = lane + 64; c < nc; c += 32) {  // contexts beyond 64 chunks
        const float2 m2 = __ldcg(reinterpret_cast<const float2*>(a.ws_ml) + head_base + (int64_t)c * d.row_cap + r);
        w_c[c] = m2.x; wl_c[c] = m2.y;
        M = fmaxf(M, m2.x);
    }
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    __syncwarp();
    for (int c = lane; c < nc; c += 32) {
        const float mc = w_c[c];
        const float f = mc == -INFINITY ? 0.f : expf(mc - M);
        w_c[c] = f; wl_c[c] = f * wl_c[c];
    }
    __syncwarp();
    float den = 0.f;
    for (int c = 0; c < nc; ++c) den += wl_c[c];  // ascending order, the same in every lane
    if (lane < HD / 4) {
        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int u = 0; u < 16; ++u) {
            if (u < nc) {
                const float f = w_c[u];
                num.x += f * p0[u].x; num.y += f * p0[u].y; num.z += f * p0[u].z; num.w += f * p0[u].w;
            }
        }
        for (int c = 16; c < nc; c += 16) {  // sixteen partials requested together
            float4 p[16];
#pragma unroll
            for (int u = 0; u < 16; ++u)
                if (c + u < nc) p[u] = __ldcg(src + (int64_t)(c + u) * d.row_cap * (HD / 4));
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                if (c + u < nc) {
                    const float f = w_c[c + u];
                    num.x += f * p[u].x; num.y += f * p[u].y; num.z += f * p[u].z; num.w += f * p[u].w;
                }
            }
        }
        const int64_t col = (int64_t)head * HD + lane * 4;
        store_act(a.attn_out, kActSplit, d.row_cap, r, col, d.hd_total, num.x / den);
        store_act(a.attn_out, kActSplit, d.row_cap, r, col + 1, d.hd_total, num.y / den);
        store_act(a.attn_out, kActSplit, d.row_cap, r, col + 2, d.hd_total, num.z / den);
        store_act(a.attn_out, kActSplit, d.row_cap, r, col + 3, d.hd_total, num.w / den);
    }
    if (lane == 0) LLMA_STAMP_MINMAX(stp, 6);
}

constexpr size_t kAttnPad = 0;  // extra shared memory per CTA (a knob for the number of CTAs per SM)

cudaError_t init_attention_mma() {
    cudaError_t e = cudaFuncSetAttribute(attention_mma_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(AttnSmem<128>::kBytes + 1024 + kAttnPad));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attention_mma_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(AttnSmem<128>::kBytes + 1024 + kAttnPad));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attention_mma_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(AttnSmem<64>::kBytes + 1024));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attention_mma_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(AttnSmem<64>::kBytes + 1024));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attention_long_kernel<128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(AttnSmem<128>::kBytes + 1024));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attention_long_kernel<128, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(AttnSmem<128>::kBytes + 1024));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attention_long_kernel<64, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(AttnSmem<64>::kBytes + 1024));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(attention_long_kernel<64, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)(AttnSmem<64>::kBytes + 1024));
}

void launch_attention_mma(cudaStream_t st, const AttnArgs& a, const CUtensorMap& map_k, const CUtensorMap& map_v) {
    dim3 grid(a.n_chunks, a.dims.n_heads, a.dims.max_batch);
    dim3 mgrid(a.dims.n_heads, (a.n_rows + 3) / 4);
    const size_t msmem = (size_t)8 * a.n_chunks * sizeof(float);
    if (!a.prompt && a.tiles > 1) {  // long contexts, many sequences: several tiles per CTA
        if (a.dims.head_dim == 128) {
            if (a.tiles == 4) launch_pdl(st, true, grid, dim3(128), AttnSmem<128>::kBytes + 1024, attention_long_kernel<128, 4>, a, map_k, map_v);
            else launch_pdl(st, true, grid, dim3(128), AttnSmem<128>::kBytes + 1024, attention_long_kernel<128, 2>, a, map_k, map_v);
            launch_pdl(st, true, mgrid, dim3(128), msmem, attention_merge_kernel<128>, a);
        } else {
            if (a.tiles == 4) launch_pdl(st, true, grid, dim3(128), AttnSmem<64>::kBytes + 1024, attention_long_kernel<64, 4>, a, map_k, map_v);
            else launch_pdl(st, true, grid, dim3(128), AttnSmem<64>::kBytes + 1024, attention_long_kernel<64, 2>, a, map_k, map_v);
            launch_pdl(st, true, mgrid, dim3(128), msmem, attention_merge_kernel<64>, a);
        }
        return;
    }
    if (a.dims.head_dim == 128) {
        if (a.prompt) launch_pdl(st, true, grid, dim3(128), AttnSmem<128>::kBytes + 1024 + kAttnPad, attention_mma_kernel<128, true>, a, map_k, map_v);
        else launch_pdl(st, true, grid, dim3(128), AttnSmem<128>::kBytes + 1024 + kAttnPad, attention_mma_kernel<128, false>, a, map_k, map_v);
        launch_pdl(st, true, mgrid, dim3(128), msmem, attention_merge_kernel<128>, a);
    } else {
        if (a.prompt) launch_pdl(st, true, grid, dim3(128), AttnSmem<64>::kBytes + 1024, attention_mma_kernel<64, true>, a, map_k, map_v);
        else launch_pdl(st, true, grid, dim3(128), AttnSmem<64>::kBytes + 1024, attention_mma_kernel<64, false>, a, map_k, map_v);
        launch_pdl(st, true, mgrid, dim3(128), msmem, attention_merge_kernel<64>, a);
    }
}

}  // namespace llma
