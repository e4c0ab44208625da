// Backward of the LTE prefill attention on the tcgen05 tensor cores (Section 3.1.2), bf16, d = 64 or 128.
//
// Two kernels, both in gather form (no floating-point atomics, deterministic):
//
// dq kernel   one CTA per 128-query tile, the same key/value tile walk as the forward kernel (window tiles by
//             TMA, retained tiles gathered with cp.async).  Per 64-key tile:
//               S = Q K^T and dP = dO V^T          tcgen05.mma into TMEM
//               P = exp2(S c2 - L2_i),  dS = P (dP - delta_i) scale   by the thread owning row i (no online softmax:
//               the forward's logsumexp fixes the normalisation), written as bf16 into swizzled shared memory
//               dQ += dS K                          tcgen05.mma, K tile as the MN-major operand, accumulated in TMEM
//             delta_i = <dO_i, O_i> is computed by the same thread at the start and also written out for the second kernel.
//
// dkv kernel  one CTA per 128-key tile: the contiguous keys of a window tile, or 128 entries of the retained list
//             (their K/V rows gathered once).  It walks the 64-query blocks that can see those keys:
//               S^T = K Q^T and dP^T = V dO^T       tcgen05.mma (keys on the M side)
//               P^T, dS^T                           by the thread owning the key row; L2 and delta of the block's
//                                                   64 queries are read from shared memory
//               dV += P^T dO,  dK += dS^T Q         tcgen05.mma with the dO / Q block as MN-major operand
//             and finishes with Eq. 6's inner product <v_j, dV_j> per key from the fp32 accumulators.  Window tiles
//             write dK, dV of their keys; retained tiles write their far-query share to scratch, which a small merge
//             kernel adds row by row (each key appears once in the list, so the sum order is fixed).
#include "tc_common.cuh"

namespace lte {

__device__ StatusWord g_bwd_status = LTE_STATUS_INIT;

namespace {

using namespace tc;
__device__ __forceinline__ void bwait(uint32_t bar, uint32_t parity, int code) { mbar_wait_s(bar, parity, code, &g_bwd_status); }
__device__ __forceinline__ void group_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

constexpr int BM = 128, BN = 64, NTHREADS = 160, NST = 3;      // 3 stages for every streamed tile
constexpr float kLog2e = 1.4426950408889634f;

template <int D> struct SmemQ {                                // dq kernel
    static constexpr int SUB = D / 64;
    // d = 128 runs one CTA per SM (shared memory), so tensor memory has room for two S / dP buffers: the products of tile
    // t+1 are in flight while the row threads work on tile t, which needs a fourth key / value stage
    static constexpr bool DB = D == 128;
    static constexpr int NS = DB ? 4 : 3;
    static constexpr int QTILE = BM * D * 2, KVTILE = BN * D * 2;
    static constexpr int OFF_Q = 0, OFF_DO = QTILE, OFF_K = 2 * QTILE, OFF_V = OFF_K + NS * KVTILE;
    static constexpr int OFF_DS = OFF_V + NS * KVTILE;         // [128][64] bf16
    static constexpr int OFF_BAR = OFF_DS + BM * BN * 2;
    static constexpr int OFF_IDX = OFF_BAR + 128;
    static constexpr int BYTES = OFF_IDX + 512;
    // d = 64:  S [0,64)  dP [64,128)  dQ [128,192);   d = 128:  S, dP of buffer b at 128 b, 128 b + 64;  dQ [256,384)
    static constexpr uint32_t TMEM_COLS = DB ? 512 : 256;
};

template <int D>
__global__ void __launch_bounds__(NTHREADS, D == 64 ? 2 : 1)
bwd_dq_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmDO,
                 const __grid_constant__ CUtensorMap tmO, const __grid_constant__ CUtensorMap tmDQ,
                 const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __nv_bfloat16* __restrict__ kg, const __nv_bfloat16* __restrict__ vg,
                 const __nv_bfloat16* __restrict__ og, const __nv_bfloat16* __restrict__ dog,
                 const float* __restrict__ lse, const int32_t* __restrict__ idx, const int32_t* __restrict__ cnt,
                 __nv_bfloat16* __restrict__ dq, float* __restrict__ delta, int Tlen, int W, int R, float scale, int G, int dg)
{
    // dg = the head dimension in memory: D, or 32 for the d = 64 kernel on d = 32 data (the tensor maps then fill the upper
    // half of every tile row with zeros on the way in and clip it on the way out; the gathers zero-fill the same columns)
    using S = SmemQ<D>;
    constexpr int SUB = S::SUB;
    constexpr bool DB = S::DB;
    constexpr int NS = S::NS;
    constexpr uint32_t DP_COL = BN, DQ_COL = DB ? 4 * BN : 2 * BN;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 1023u) != 0) { if (threadIdx.x == 0) atomicExch(&g_bwd_status.code, 9); return; }
    const uint32_t sQ = base + S::OFF_Q, sDO = base + S::OFF_DO, sK = base + S::OFF_K, sV = base + S::OFF_V;
    const uint32_t sDS = base + S::OFF_DS;
    const uint32_t bar_q = base + S::OFF_BAR, bar_k0 = bar_q + 8, bar_v0 = bar_q + 40, bar_s0 = bar_q + 72;   // 4, 4, 2 slots
    const uint32_t bar_g0 = bar_q + 88, bar_p = bar_q + 104, bar_pv = bar_q + 112, tmem_slot = bar_q + 120;
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_raw + S::OFF_BAR + 120);
    volatile int* s_idx = reinterpret_cast<volatile int*>(smem_raw + S::OFF_IDX);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.y, bhk = bh / G;                   // query head; its key/value head (grouped queries: G per head)
    const int i0 = blockIdx.x * BM;
    const int i_hi = min(i0 + BM - 1, Tlen - 1);
    const int j_start = max(i0 - W + 1, 0);
    const int n_win = (i_hi - j_start + 1 + BN - 1) / BN;
    const int32_t* id = idx + (size_t)bhk * R;

    if (tid == 0) {
        mbar_init(bar_q, 1);
#pragma unroll
        for (int s2 = 0; s2 < NS; ++s2) { mbar_init(bar_k0 + 8 * s2, 1); mbar_init(bar_v0 + 8 * s2, 1); }
        mbar_init(bar_s0, 1); mbar_init(bar_s0 + 8, 1);
        mbar_init(bar_g0, 128); mbar_init(bar_g0 + 8, 128);
        mbar_init(bar_p, 128); mbar_init(bar_pv, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) tmem_alloc(tmem_slot, S::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;
    pdl_launch_dependents();
    pdl_wait();                                                // everything above ran beside the previous kernel's tail (see launch_pdl)
    const int n_ret = cnt[bhk];

    if (warp == 4) {
        // =================================== control warp (one lane) ========================================
        int n_tiles = n_win;                                   // + the retained tiles, counted once the first loads are on their way
        // The whole warp walks the loop and waits on the barriers; only the TMA / tcgen05 instructions are guarded by the
        // lane test, so that addresses and descriptors are computed in convergent code (cheaper to issue).
        const bool leader = lane == 0;
        {
            constexpr uint32_t IDESC_S = instr_desc(BM, BN, false);
            constexpr uint32_t IDESC_Q = instr_desc(BM, D, true);
            const uint32_t q_lo = desc_lo(sQ, 16), do_lo = desc_lo(sDO, 16), k_lo = desc_lo(sK, 16), v_lo = desc_lo(sV, 16);
            const uint32_t ds_lo = desc_lo(sDS, 16), kmn_lo = desc_lo(sK, 8192);
            uint32_t k_phase = 0, v_phase = 0, g_waited = 0;
            auto tma_kv = [&](int t, bool is_v) {
                const int st = t % NS;
                const uint32_t dst = (is_v ? sV : sK) + st * S::KVTILE;
                const uint32_t bar = (is_v ? bar_v0 : bar_k0) + 8 * st;
                const int y = j_start + t * BN;
                if (leader) {
                    mbar_expect_tx(bar, S::KVTILE);
#pragma unroll
                    for (int sb = 0; sb < SUB; ++sb) tma_load_3d(dst + sb * 8192, is_v ? &tmV : &tmK, sb * 64, y, bhk, bar);
                }
            };
            auto need_g = [&](uint32_t phase) {
                while (g_waited <= phase) { bwait(bar_g0 + 8 * (g_waited & 1), (g_waited >> 1) & 1, 10); ++g_waited; }
            };
            auto wait_kv = [&](int t) {
                if (t < n_win) {
                    const int st = t % NS;
                    bwait(bar_k0 + 8 * st, (k_phase >> st) & 1u, 2); k_phase ^= 1u << st;
                    bwait(bar_v0 + 8 * st, (v_phase >> st) & 1u, 4); v_phase ^= 1u << st;
                }
            };
            auto mma_s_dp = [&](int t) {
                const uint32_t so = (uint32_t)(t % NS) * (S::KVTILE >> 4);
                const uint32_t sbuf = DB ? (uint32_t)(t & 1) * (2 * BN) : 0u;
                if (leader) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        umma(tmem + sbuf, desc64(q_lo + (kk >> 2) * 1024 + (kk & 3) * 2, kDescHi),
                             desc64(k_lo + so + (kk >> 2) * 512 + (kk & 3) * 2, kDescHi), IDESC_S, kk > 0);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        umma(tmem + sbuf + DP_COL, desc64(do_lo + (kk >> 2) * 1024 + (kk & 3) * 2, kDescHi),
                             desc64(v_lo + so + (kk >> 2) * 512 + (kk & 3) * 2, kDescHi), IDESC_S, kk > 0);
                    umma_commit(bar_s0 + (DB ? 8 * (t & 1) : 0));
                }
                __syncwarp();
            };

            // d = 64: the O tile rides along into the (still unused) dS buffer, for delta = <dO, O>
            if (leader) {
                mbar_expect_tx(bar_q, (D == 64 ? 3 : 2) * S::QTILE);
#pragma unroll
                for (int sb = 0; sb < SUB; ++sb) {
                    tma_load_3d(sQ + sb * 16384, &tmQ, sb * 64, i0, bh, bar_q);
                    tma_load_3d(sDO + sb * 16384, &tmDO, sb * 64, i0, bh, bar_q);
                }
                if (D == 64) tma_load_3d(sDS, &tmO, 0, i0, bh, bar_q);
            }
            for (int t = 0; t < NS && t < n_win; ++t) { tma_kv(t, false); tma_kv(t, true); }
            {
                // retained entries visible to the tile's last row (idx ascending => a prefix): read while the loads fly
                int nv_max = 0;
                const int lim = i_hi - W;
                for (int e0 = 0; e0 < n_ret; e0 += 32) {
                    const int e = e0 + lane < n_ret ? id[e0 + lane] : 0x7fffffff;
                    const unsigned bal = __ballot_sync(0xffffffffu, e <= lim);
                    nv_max += __popc(bal);
                    if (bal != 0xffffffffu) break;
                }
                n_tiles = n_win + (nv_max + BN - 1) / BN;
            }
            bwait(bar_q, 0, 1);                                // (tile 0 is always a window tile: no gather to wait for)
            wait_kv(0);
            tc_fence_after();
            mma_s_dp(0);
            if (DB && n_tiles > 1) {                           // two buffers: tile 1 follows at once (prologue gathers: phase 0)
                need_g(0);
                wait_kv(1);
                tc_fence_after();
                mma_s_dp(1);
            }
            for (int t = 0; t < n_tiles; ++t) {
                bwait(bar_p, t & 1, 7);                        // dS(t) is in shared memory; its S / dP buffer is free
                tc_fence_after();
                // one buffer: the next tile's S, dP first: the row threads wait for those, while dQ of this tile is only
                // needed before the dS buffer is rewritten a tile later
                if (!DB && t + 1 < n_tiles) {
                    need_g(t + 1);
                    wait_kv(t + 1);
                    mma_s_dp(t + 1);
                }
                {
                    const uint32_t kb = kmn_lo + (uint32_t)(t % NS) * (S::KVTILE >> 4);
                    if (leader) {
#pragma unroll
                        for (int kk = 0; kk < BN / 16; ++kk)
                            umma(tmem + DQ_COL, desc64(ds_lo + kk * 2, kDescHi), desc64(kb + kk * 128, kDescHi), IDESC_Q,
                                 (t > 0 || kk > 0) ? 1u : 0u);
                        umma_commit(bar_pv);
                    }
                    __syncwarp();
                }
                // two buffers: the row threads are already on tile t+1; S, dP of tile t+2 go into the buffer tile t has left.
                // Its gathers were committed in tile t-1 and are covered by the arrival at the top of tile t+1.
                if (DB && t + 2 < n_tiles) {
                    need_g(t + 1);
                    wait_kv(t + 2);
                    tc_fence_after();
                    mma_s_dp(t + 2);
                }
                // dQ(t-1) has completed (the softmax warps waited for it before producing dS(t)): its key stage and
                // the value stage of tile t-1 can take window tile t-1+NS
                if (t >= 1 && t - 1 + NS < n_win) { tma_kv(t - 1 + NS, false); tma_kv(t - 1 + NS, true); }
            }
        }
    } else {
        // =================================== softmax warps ==================================================
        const int i = i0 + tid;
        const int ic = min(i, Tlen - 1);
        // delta_i = <dO_i, O_i>, L2_i = lse_i * log2(e).  d = 64: both rows are in shared memory (the TMA tiles of dO and
        // O, 128-byte swizzle: chunk c of row r sits at chunk position c ^ (r & 7)); d = 128: from global memory.
        float dl = 0.f;
        const float L2 = lse[(size_t)bh * Tlen + ic] * kLog2e;
        if (D == 64) {
            bwait(bar_q, 0, 12);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint32_t off = tid * 128 + ((c ^ (tid & 7)) << 4);
                uint32_t aw[4], bw[4];
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(aw[0]), "=r"(aw[1]), "=r"(aw[2]), "=r"(aw[3]) : "r"(sDS + off));
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(bw[0]), "=r"(bw[1]), "=r"(bw[2]), "=r"(bw[3]) : "r"(sDO + off));
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    dl = fmaf(__uint_as_float(aw[u] << 16), __uint_as_float(bw[u] << 16), dl);
                    dl = fmaf(__uint_as_float(aw[u] & 0xffff0000u), __uint_as_float(bw[u] & 0xffff0000u), dl);
                }
            }
        } else {
            const uint4* orow = reinterpret_cast<const uint4*>(og + ((size_t)bh * Tlen + ic) * D);
            const uint4* grow = reinterpret_cast<const uint4*>(dog + ((size_t)bh * Tlen + ic) * D);
#pragma unroll 4
            for (int c = 0; c < D / 8; ++c) {
                const uint4 a = orow[c], b = grow[c];
                const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    dl = fmaf(__uint_as_float(aw[u] << 16), __uint_as_float(bw[u] << 16), dl);
                    dl = fmaf(__uint_as_float(aw[u] & 0xffff0000u), __uint_as_float(bw[u] & 0xffff0000u), dl);
                }
            }
        }
        if (i < Tlen) delta[(size_t)bh * Tlen + i] = dl;

        // retained entries visible to this row: rows of a warp are consecutive and the list is ascending, so the count is
        // #{idx <= lim of lane 0} plus the entries between the warp's first limit and this lane's (a 31-bit map)
        const int lim = ic - W, lim_max = i_hi - W;
        const int lim0 = __shfl_sync(0xffffffffu, lim, 0), lim31 = __shfl_sync(0xffffffffu, lim, 31);
        int nvis = 0, nv_max = 0;
        {
            uint32_t bits = 0;
            for (int e0 = 0; e0 < n_ret; e0 += 128) {
                int e[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) e[u] = e0 + u * 32 + lane < n_ret ? id[e0 + u * 32 + lane] : 0x7fffffff;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    nvis += __popc(__ballot_sync(0xffffffffu, e[u] <= lim0));
                    nv_max += __popc(__ballot_sync(0xffffffffu, e[u] <= lim_max));
                    const bool in = e[u] > lim0 && e[u] <= lim31;
                    bits |= __reduce_or_sync(0xffffffffu, in ? 1u << (e[u] - lim0 - 1) : 0u);
                }
                if (__shfl_sync(0xffffffffu, e[3], 31) > lim_max) break;
            }
            nvis += __popc(bits & ((1u << (lim - lim0)) - 1u));
        }
        const int n_tiles = n_win + (nv_max + BN - 1) / BN;

        const int g_row = tid >> 3, g_sub = tid & 7;
        auto gather_rows = [&](int t, int (&rows4)[4]) {
#pragma unroll
            for (int ps = 0; ps < 4; ++ps) {
                const int e = (t - n_win) * BN + ps * 16 + g_row;
                rows4[ps] = (t >= n_win && t < n_tiles && e < nv_max) ? id[e] : -1;
            }
        };
        auto gather_issue = [&](int t, bool is_v, const int (&rows4)[4]) {
            if (t >= n_win && t < n_tiles) {
                const uint32_t dst = (is_v ? sV : sK) + (t % NS) * S::KVTILE;
#pragma unroll
                for (int ps = 0; ps < 4; ++ps) {
                    const int row = ps * 16 + g_row;
                    const bool ok = rows4[ps] >= 0;
                    const __nv_bfloat16* src = (is_v ? vg : kg) + ((size_t)bhk * Tlen + (ok ? rows4[ps] : 0)) * dg;
#pragma unroll
                    for (int c = g_sub; c < D / 8; c += 8) {
                        const uint32_t off = (c >> 3) * 8192 + row * 128 + (((c & 7) ^ (row & 7)) << 4);
                        const bool real = ok && c * 8 < dg;
                        cp_async16(dst + off, src + (real ? c * 8 : 0), real ? 16u : 0u);
                    }
                }
            }
        };
        {
            int rows4[4];
            for (int t = 0; t < NS; ++t) { gather_rows(t, rows4); gather_issue(t, false, rows4); gather_issue(t, true, rows4); }
            cp_async_commit();
            cp_async_commit();                                 // empty group: the wait at the top of tile 0 then covers the one above
        }
        const float c2 = scale * kLog2e;
        const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;

        for (int t = 0; t < n_tiles; ++t) {
            int rn[4];
            gather_rows(t - 1 + NS, rn);                       // retained tile that goes into the stage of tile t-1
            cp_async_wait<1>();                                // every gather but the latest tile's has landed
            fence_proxy_async();
            mbar_arrive(bar_g0 + 8 * (t & 1));

            int c_lo, c_hi;
            if (t < n_win) {
                const int jt0 = j_start + t * BN;
                c_lo = max(i - W + 1, 0) - jt0;
                c_hi = i - jt0;
            } else {
                c_lo = 0;
                c_hi = nvis - (t - n_win) * BN - 1;
            }
            const int u_lo = __shfl_sync(0xffffffffu, c_lo, 0), u_hi = __shfl_sync(0xffffffffu, c_hi, 31);

            bwait(bar_s0 + (DB ? 8 * (t & 1) : 0), DB ? (t >> 1) & 1 : t & 1, 3);   // S(t), dP(t) are in TMEM
            tc_fence_after();
            const uint32_t sbuf = DB ? (uint32_t)(t & 1) * (2 * BN) : 0u;
            uint32_t pk[32];                                   // dS row as 64 bf16
            const uint64_t c2_2 = pack2(c2, c2), nl2_2 = pack2(-L2, -L2), scale_2 = pack2(scale, scale), ndls_2 = pack2(-dl * scale, -dl * scale);
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                const bool act = cb * 32 <= u_hi && cb * 32 + 31 >= u_lo;
                if (act) {
                    uint32_t rs[32], rp[32];
                    tmem_ld32(tmem + lane_base + sbuf + cb * 32, rs);
                    tmem_ld32(tmem + lane_base + sbuf + DP_COL + cb * 32, rp);
                    tmem_wait_ld();
                    // validity bits of this row's 32 columns; the arithmetic runs on packed fp32 pairs
                    const int a = min(max(c_lo - cb * 32, 0), 32), b2 = min(max(c_hi - cb * 32 + 1, 0), 32);
                    const uint32_t below_b = b2 >= 32 ? 0xffffffffu : ((1u << b2) - 1u);
                    const uint32_t below_a = a >= 32 ? 0xffffffffu : ((1u << a) - 1u);
                    const uint32_t vm = b2 > a ? (below_b & ~below_a) : 0u;
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        float x0, x1, d0, d1;
                        unpack2(fma2(pack2(__uint_as_float(rs[c]), __uint_as_float(rs[c + 1])), c2_2, nl2_2), x0, x1);
                        const uint64_t g2 = fma2(pack2(__uint_as_float(rp[c]), __uint_as_float(rp[c + 1])), scale_2, ndls_2);   // (dP - delta) scale
                        unpack2(mul2(pack2(fast_exp2(x0), fast_exp2(x1)), g2), d0, d1);
                        __nv_bfloat162 h = __floats2bfloat162_rn((vm & (1u << c)) ? d0 : 0.f, (vm & (2u << c)) ? d1 : 0.f);
                        pk[cb * 16 + (c >> 1)] = *reinterpret_cast<uint32_t*>(&h);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 16; ++c) pk[cb * 16 + c] = 0u;
                }
            }
            // dQ(t-1) must be done before dS is overwritten; its key stage (and the value stage) are then free
            if (t > 0) { bwait(bar_pv, (t - 1) & 1, 4); tc_fence_after(); }
            if (t > 0) { gather_issue(t - 1 + NS, false, rn); gather_issue(t - 1 + NS, true, rn); }
            cp_async_commit();
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                const uint32_t dst = sDS + tid * 128 + ((ch ^ (tid & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[4 * ch]), "r"(pk[4 * ch + 1]),
                             "r"(pk[4 * ch + 2]), "r"(pk[4 * ch + 3]) : "memory");
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar_p);
        }
        bwait(bar_pv, (n_tiles - 1) & 1, 5);
        tc_fence_after();
        // ---- epilogue: dQ (the softmax scale is already folded into dS) ------------------------------------
        if (D == 64) {
            // the rows go into the (now idle) dS buffer in the swizzled layout and leave as one tile store per warp
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                uint32_t q4[32];
                tmem_ld32(tmem + lane_base + DQ_COL + cb * 32, q4);
                tmem_wait_ld();
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    uint32_t w4[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(q4[g * 8 + 2 * u]), __uint_as_float(q4[g * 8 + 2 * u + 1]));
                        w4[u] = *reinterpret_cast<uint32_t*>(&h);
                    }
                    const int ch = cb * 4 + g;
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sDS + tid * 128 + ((ch ^ (tid & 7)) << 4)),
                                 "r"(w4[0]), "r"(w4[1]), "r"(w4[2]), "r"(w4[3]) : "memory");
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0 && i0 + warp * 32 < Tlen) {
                tma_store_3d(&tmDQ, sDS + warp * 4096, 0, i0 + warp * 32, bh);
                bulk_commit();
                bulk_wait_read0();                             // the buffer is released with the CTA
            }
        } else {
            __nv_bfloat16* qrow = dq + ((size_t)bh * Tlen + i) * D;
#pragma unroll
            for (int cb = 0; cb < D / 32; ++cb) {
                uint32_t q4[32];
                tmem_ld32(tmem + lane_base + DQ_COL + cb * 32, q4);
                tmem_wait_ld();
                if (i < Tlen) {
#pragma unroll
                    for (int c = 0; c < 32; c += 8) {
                        uint32_t w4[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(q4[c + 2 * u]), __uint_as_float(q4[c + 2 * u + 1]));
                            w4[u] = *reinterpret_cast<uint32_t*>(&h);
                        }
                        *reinterpret_cast<uint4*>(qrow + cb * 32 + c) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, S::TMEM_COLS);
}


// ================================================ dkv kernel =====================================================
template <int D> struct SmemK {
    static constexpr int SUB = D / 64;
    // d = 128 runs one CTA per SM and has the TMEM columns for two S^T / dP^T buffers: block t+2's products are issued
    // while the key threads work on block t+1, which takes one more stage of query blocks in flight
    static constexpr bool DB = D == 128;
    static constexpr int NSTK = DB ? 4 : 3;
    static constexpr int KTILE = 128 * D * 2, QBLK = 64 * D * 2;
    static constexpr int OFF_K = 0, OFF_V = KTILE, OFF_Q = 2 * KTILE, OFF_DO = OFF_Q + NSTK * QBLK;
    static constexpr int OFF_PT = OFF_DO + NSTK * QBLK;        // [128][64] bf16
    static constexpr int OFF_DST = OFF_PT + 128 * 64 * 2;      // [128][64] bf16
    static constexpr int OFF_COL = OFF_DST + 128 * 64 * 2;     // L2[64], delta[64] of the current query block
    static constexpr int OFF_BAR = OFF_COL + 512;
    static constexpr int BYTES = OFF_BAR + 128;
    // d = 64: S^T [0,64) dP^T [64,128) dV [128,192) dK [192,256); d = 128: S^T, dP^T of even blocks [0,128), of odd blocks
    // [128,256), dV [256,384), dK [384,512)
    static constexpr uint32_t TMEM_COLS = D == 64 ? 256 : 512;
};

template <int D, bool F32OUT>
__global__ void __launch_bounds__(NTHREADS, D == 64 ? 2 : 1)
bwd_dkv_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                  const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmDO,
                  const __grid_constant__ CUtensorMap tmDK, const __grid_constant__ CUtensorMap tmDV,
                  const __nv_bfloat16* __restrict__ kg, const __nv_bfloat16* __restrict__ vg,
                  const float* __restrict__ lse, const float* __restrict__ delta, const int32_t* __restrict__ idx,
                  const int32_t* __restrict__ cnt, __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                  float* __restrict__ dk32, float* __restrict__ dv32, float* __restrict__ dr_win,
                  float* __restrict__ dk_ret, float* __restrict__ dv_ret, float* __restrict__ dr_ret, int n_wt, int Tlen,
                  int W, int R, float scale, int G, int dg)
{
    using S = SmemK<D>;
    constexpr int SUB = S::SUB;
    constexpr bool DB = S::DB;
    constexpr int NSTK = S::NSTK;
    constexpr uint32_t DP_COL = 64, DV_COL = DB ? 256 : 128, DK_COL = DV_COL + D;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 1023u) != 0) { if (threadIdx.x == 0) atomicExch(&g_bwd_status.code, 9); return; }
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // the retained tiles walk many more query blocks than the window tiles: they take the lowest block numbers so
    // that they start first and do not form the tail of the launch
    const int n_rt = (int)gridDim.x - n_wt;
    const int lin = blockIdx.y * gridDim.x + blockIdx.x, tot_ret = n_rt * (int)gridDim.y;
    const bool is_ret = lin < tot_ret;
    const int bh = is_ret ? lin / n_rt : (lin - tot_ret) / n_wt;
    const int tile = is_ret ? lin % n_rt : (lin - tot_ret) % n_wt;
    const uint32_t sK = base + S::OFF_K, sV = base + S::OFF_V, sQ = base + S::OFF_Q, sDO = base + S::OFF_DO;
    const uint32_t sPT = base + S::OFF_PT, sDST = base + S::OFF_DST;
    float* s_col = reinterpret_cast<float*>(smem_raw + S::OFF_COL);
    const uint32_t bar_kv = base + S::OFF_BAR, bar_q0 = bar_kv + 8, bar_s0 = bar_kv + 40, bar_g = bar_kv + 56;
    const uint32_t bar_p = bar_kv + 64, bar_pv = bar_kv + 72, tmem_slot = bar_kv + 80;
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_raw + S::OFF_BAR + 80);

    if (tid == 0) {
        mbar_init(bar_kv, 1);
#pragma unroll
        for (int s2 = 0; s2 < NSTK; ++s2) mbar_init(bar_q0 + 8 * s2, 1);
        mbar_init(bar_s0, 1); mbar_init(bar_s0 + 8, 1); mbar_init(bar_g, 128); mbar_init(bar_p, 128); mbar_init(bar_pv, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) tmem_alloc(tmem_slot, S::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;
    pdl_launch_dependents();
    pdl_wait();                                                // everything above ran beside the previous kernel's tail (see launch_pdl)
    const int n_ret = cnt[bh];
    const int32_t* id = idx + (size_t)bh * R;
    const int j0 = is_ret ? 0 : tile * 128;                    // window tile: first key
    const int e0 = is_ret ? tile * 128 : 0;                    // retained tile: first list entry
    if (is_ret && e0 >= n_ret) {                               // nothing retained in this slice of the list
        if (warp == 4) tmem_dealloc(tmem, S::TMEM_COLS);
        return;
    }

    // query blocks that can see the tile
    int ib_start, n_blk;
    if (!is_ret) {
        ib_start = j0;
        const int i_end = min(Tlen - 1, j0 + 127 + W - 1);
        n_blk = (i_end - ib_start) / 64 + 1;
    } else {
        const int first = id[e0] + W;                          // the oldest entry's first far query
        ib_start = (first / 64) * 64;
        n_blk = first <= Tlen - 1 ? (Tlen - 1 - ib_start) / 64 + 1 : 0;
    }
    // grouped queries: the G query heads of this key/value head walk the same query blocks one after the other and
    // accumulate into the same dK, dV; walk step t is block t % n_pos of query head bh G + t / n_pos
    const int n_pos = n_blk;
    n_blk *= G;

    if (warp == 4) {
        // (the whole warp walks the loop and waits; only the TMA / tcgen05 instructions are guarded by the lane test)
        const bool leader = lane == 0;
        if (n_blk > 0) {
            constexpr uint32_t IDESC_S = instr_desc(128, 64, false);
            constexpr uint32_t IDESC_O = instr_desc(128, D, true);
            const uint32_t k_lo = desc_lo(sK, 16), v_lo = desc_lo(sV, 16), q_lo = desc_lo(sQ, 16), do_lo = desc_lo(sDO, 16);
            const uint32_t pt_lo = desc_lo(sPT, 16), dst_lo = desc_lo(sDST, 16);
            const uint32_t qmn_lo = desc_lo(sQ, 8192), domn_lo = desc_lo(sDO, 8192);
            uint32_t q_phase = 0;
            auto tma_blk = [&](int t) {
                const int st = t % NSTK;
                const uint32_t bar = bar_q0 + 8 * st;
                const int y = ib_start + (t % n_pos) * 64, bhq = bh * G + t / n_pos;
                if (leader) {
                    mbar_expect_tx(bar, 2 * S::QBLK);
#pragma unroll
                    for (int sb = 0; sb < SUB; ++sb) {
                        tma_load_3d(sQ + st * S::QBLK + sb * 8192, &tmQ, sb * 64, y, bhq, bar);
                        tma_load_3d(sDO + st * S::QBLK + sb * 8192, &tmDO, sb * 64, y, bhq, bar);
                    }
                }
            };
            auto wait_blk = [&](int t) {
                const int st = t % NSTK;
                bwait(bar_q0 + 8 * st, (q_phase >> st) & 1u, 2); q_phase ^= 1u << st;
            };
            auto mma_s_dp = [&](int t) {
                const uint32_t so = (uint32_t)(t % NSTK) * (S::QBLK >> 4);
                const uint32_t tb = tmem + (DB ? (uint32_t)(t & 1) * 128u : 0u);
                if (leader) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        umma(tb, desc64(k_lo + (kk >> 2) * 1024 + (kk & 3) * 2, kDescHi),
                             desc64(q_lo + so + (kk >> 2) * 512 + (kk & 3) * 2, kDescHi), IDESC_S, kk > 0);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        umma(tb + DP_COL, desc64(v_lo + (kk >> 2) * 1024 + (kk & 3) * 2, kDescHi),
                             desc64(do_lo + so + (kk >> 2) * 512 + (kk & 3) * 2, kDescHi), IDESC_S, kk > 0);
                    umma_commit(DB ? bar_s0 + 8 * (t & 1) : bar_s0);
                }
                __syncwarp();
            };
            if (!is_ret && leader) {
                mbar_expect_tx(bar_kv, 2 * S::KTILE);
#pragma unroll
                for (int sb = 0; sb < SUB; ++sb) {
                    tma_load_3d(sK + sb * 16384, &tmK, sb * 64, j0, bh, bar_kv);
                    tma_load_3d(sV + sb * 16384, &tmV, sb * 64, j0, bh, bar_kv);
                }
            }
            for (int t = 0; t < NSTK && t < n_blk; ++t) tma_blk(t);
            if (!is_ret) bwait(bar_kv, 0, 1); else bwait(bar_g, 0, 10);   // the tile's own K/V rows are in shared memory
            wait_blk(0);
            tc_fence_after();
            mma_s_dp(0);
            if (DB && n_blk > 1) { wait_blk(1); mma_s_dp(1); }
            for (int t = 0; t < n_blk; ++t) {
                bwait(bar_p, t & 1, 7);                        // P^T(t), dS^T(t) are in shared memory
                tc_fence_after();
                // one buffer: the next block's S^T, dP^T first (the key threads wait for those, while dV, dK of this block
                // are only needed before the operand buffers are rewritten a block later); two buffers: the next block's
                // products are already there, so dV, dK go first and block t+2's products take the buffer of block t,
                // which the key threads have read out
                if (!DB && t + 1 < n_blk) { wait_blk(t + 1); mma_s_dp(t + 1); }
                {
                    const uint32_t so = (uint32_t)(t % NSTK) * (S::QBLK >> 4);
                    if (leader) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma(tmem + DV_COL, desc64(pt_lo + kk * 2, kDescHi), desc64(domn_lo + so + kk * 128, kDescHi), IDESC_O,
                                 (t > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma(tmem + DK_COL, desc64(dst_lo + kk * 2, kDescHi), desc64(qmn_lo + so + kk * 128, kDescHi), IDESC_O,
                                 (t > 0 || kk > 0) ? 1u : 0u);
                        umma_commit(bar_pv);
                    }
                    __syncwarp();
                }
                if (DB && t + 2 < n_blk) { wait_blk(t + 2); mma_s_dp(t + 2); }
                // the accumulations of block t-1 have completed (the key threads waited for them before producing
                // block t's operands): its stage can take block t-1+NSTK
                if (t >= 1 && t - 1 + NSTK < n_blk) tma_blk(t - 1 + NSTK);
            }
        }
    } else {
        // ==================================== key threads: thread r owns key row r ===========================
        const int pos = is_ret ? (e0 + tid < n_ret ? id[e0 + tid] : -1) : (j0 + tid < Tlen ? j0 + tid : -1);
        if (is_ret) {
            // this tile's K / V rows, gathered once (zero rows past the end of the list)
            const size_t rowoff = ((size_t)bh * Tlen + (pos >= 0 ? pos : 0)) * dg;   // dg: the head dimension in memory (see the dq kernel)
#pragma unroll
            for (int c = 0; c < D / 8; ++c) {
                const uint32_t off = (c >> 3) * 16384 + tid * 128 + (((c & 7) ^ (tid & 7)) << 4);
                const bool real = pos >= 0 && c * 8 < dg;
                cp_async16(sK + off, kg + rowoff + (real ? c * 8 : 0), real ? 16u : 0u);
                cp_async16(sV + off, vg + rowoff + (real ? c * 8 : 0), real ? 16u : 0u);
            }
            cp_async_commit();
            cp_async_wait<0>();
            fence_proxy_async();
            mbar_arrive(bar_g);
        }
        const float c2 = scale * kLog2e;
        const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;
        // per-column constants of the next block, fetched one block ahead: thread c < 64 holds -L2, thread 64 + c
        // -delta scale (the forms the fused multiply-adds below take).  The fetch returns the value as loaded and the
        // factor is applied a block later, where it is stored: arithmetic placed right behind the load would hold the
        // warp (which issues in order) for the whole latency of the load.
        const float* col_src = tid < 64 ? lse : delta;
        const float col_mul = tid < 64 ? -kLog2e : -scale;
        auto col_fetch = [&](int t) -> float {
            if (t >= n_blk) return 0.f;
            const int i = ib_start + (t % n_pos) * 64 + (tid & 63);
            if (i >= Tlen) return tid < 64 ? INFINITY : 0.f;                    // -L2 = -inf makes P = 0
            const size_t bhq = (size_t)bh * G + t / n_pos;
            return col_src[bhq * Tlen + i];
        };
        float col_next = col_fetch(0);

        for (int t = 0; t < n_blk; ++t) {
            group_sync();                                      // everyone is done with the previous block's constants
            s_col[tid] = col_next * col_mul;
            col_next = col_fetch(t + 1);
            group_sync();
            const int ib = ib_start + (t % n_pos) * 64;
            int c_lo, c_hi;                                    // query columns of the block this key row may be seen by
            if (pos < 0) { c_lo = 1 << 20; c_hi = -(1 << 20); }
            else if (!is_ret) { c_lo = pos - ib; c_hi = min(pos + W - 1, Tlen - 1) - ib; }
            else { c_lo = pos + W - ib; c_hi = Tlen - 1 - ib; }
            const int u_lo = __reduce_min_sync(0xffffffffu, c_lo), u_hi = __reduce_max_sync(0xffffffffu, c_hi);

            if (DB) bwait(bar_s0 + 8 * (t & 1), (t >> 1) & 1, 3);   // S^T(t), dP^T(t) are in TMEM
            else bwait(bar_s0, t & 1, 3);
            tc_fence_after();
            const uint32_t tb = tmem + lane_base + (DB ? (uint32_t)(t & 1) * 128u : 0u);
            uint32_t pp[32], pd[32];                           // P^T and dS^T rows as 64 bf16 each
            const uint64_t c2_2 = pack2(c2, c2), scale_2 = pack2(scale, scale);
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                const bool act = cb * 32 <= u_hi && cb * 32 + 31 >= u_lo;
                if (act) {
                    uint32_t rs[32], rp[32];
                    tmem_ld32(tb + cb * 32, rs);
                    tmem_ld32(tb + DP_COL + cb * 32, rp);
                    const int a = min(max(c_lo - cb * 32, 0), 32), b2 = min(max(c_hi - cb * 32 + 1, 0), 32);
                    const uint32_t below_b = b2 >= 32 ? 0xffffffffu : ((1u << b2) - 1u);
                    const uint32_t below_a = a >= 32 ? 0xffffffffu : ((1u << a) - 1u);
                    const uint32_t vm = b2 > a ? (below_b & ~below_a) : 0u;   // validity bits of this row's 32 columns
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        const int col = cb * 32 + c;
                        const float4 l4 = *reinterpret_cast<const float4*>(&s_col[col]);
                        const float4 d4 = *reinterpret_cast<const float4*>(&s_col[64 + col]);
                        // packed fp32 pairs: exponent arguments, (dP scale - delta scale), their product with P
                        float x[4], p[4], ds[4];
                        unpack2(fma2(pack2(__uint_as_float(rs[c]), __uint_as_float(rs[c + 1])), c2_2, pack2(l4.x, l4.y)), x[0], x[1]);
                        unpack2(fma2(pack2(__uint_as_float(rs[c + 2]), __uint_as_float(rs[c + 3])), c2_2, pack2(l4.z, l4.w)), x[2], x[3]);
#pragma unroll
                        for (int u = 0; u < 4; ++u) p[u] = (vm & (1u << (c + u))) ? fast_exp2(x[u]) : 0.f;
                        unpack2(mul2(pack2(p[0], p[1]), fma2(pack2(__uint_as_float(rp[c]), __uint_as_float(rp[c + 1])), scale_2, pack2(d4.x, d4.y))), ds[0], ds[1]);
                        unpack2(mul2(pack2(p[2], p[3]), fma2(pack2(__uint_as_float(rp[c + 2]), __uint_as_float(rp[c + 3])), scale_2, pack2(d4.z, d4.w))), ds[2], ds[3]);
                        __nv_bfloat162 h0 = __floats2bfloat162_rn(p[0], p[1]), h1 = __floats2bfloat162_rn(p[2], p[3]);
                        __nv_bfloat162 g0 = __floats2bfloat162_rn(ds[0], ds[1]), g1 = __floats2bfloat162_rn(ds[2], ds[3]);
                        pp[cb * 16 + (c >> 1)] = *reinterpret_cast<uint32_t*>(&h0);
                        pp[cb * 16 + (c >> 1) + 1] = *reinterpret_cast<uint32_t*>(&h1);
                        pd[cb * 16 + (c >> 1)] = *reinterpret_cast<uint32_t*>(&g0);
                        pd[cb * 16 + (c >> 1) + 1] = *reinterpret_cast<uint32_t*>(&g1);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 16; ++c) { pp[cb * 16 + c] = 0u; pd[cb * 16 + c] = 0u; }
                }
            }
            if (t > 0) { bwait(bar_pv, (t - 1) & 1, 4); tc_fence_after(); }   // the MMAs reading the old operands are done
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                const uint32_t off = tid * 128 + ((ch ^ (tid & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sPT + off), "r"(pp[4 * ch]), "r"(pp[4 * ch + 1]),
                             "r"(pp[4 * ch + 2]), "r"(pp[4 * ch + 3]) : "memory");
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sDST + off), "r"(pd[4 * ch]), "r"(pd[4 * ch + 1]),
                             "r"(pd[4 * ch + 2]), "r"(pd[4 * ch + 3]) : "memory");
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar_p);
        }
        if (n_blk > 0) { bwait(bar_pv, (n_blk - 1) & 1, 5); tc_fence_after(); }

        // ---- epilogue: dV, dK rows and Eq. 6's <v_j, dV_j> ------------------------------------------------------
        float dr = 0.f;
        const bool live = pos >= 0;
        const size_t orow = is_ret ? ((size_t)bh * R + e0 + tid) * dg : ((size_t)bh * Tlen + (live ? pos : 0)) * dg;
#pragma unroll
        for (int half2 = 0; half2 < 2; ++half2) {              // 0: dV, 1: dK
#pragma unroll
            for (int cb = 0; cb < D / 32; ++cb) {
                uint32_t a4[32];
                if (n_blk > 0) {
                    tmem_ld32(tmem + lane_base + (half2 ? DK_COL : DV_COL) + cb * 32, a4);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c) a4[c] = 0u;
                }
                if (half2 == 0) {
                    // v row of this key from the swizzled tile in shared memory
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const int ch = cb * 4 + g;             // 16-byte chunk index within the row
                        const uint4 u = *reinterpret_cast<const uint4*>(smem_raw + S::OFF_V + (ch >> 3) * 16384 + tid * 128 +
                                                                        (((ch & 7) ^ (tid & 7)) << 4));
                        const uint32_t w4[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            dr = fmaf(__uint_as_float(w4[x] << 16), __uint_as_float(a4[g * 8 + 2 * x]), dr);
                            dr = fmaf(__uint_as_float(w4[x] & 0xffff0000u), __uint_as_float(a4[g * 8 + 2 * x + 1]), dr);
                        }
                    }
                }
                if (live && cb * 32 < dg && (is_ret || F32OUT || D != 64)) {
                    if (is_ret || F32OUT) {
                        float* dst = (is_ret ? (half2 ? dk_ret : dv_ret) : (half2 ? dk32 : dv32)) + orow + cb * 32;
#pragma unroll
                        for (int c = 0; c < 32; c += 4)
                            *reinterpret_cast<float4*>(dst + c) = make_float4(__uint_as_float(a4[c]), __uint_as_float(a4[c + 1]),
                                                                              __uint_as_float(a4[c + 2]), __uint_as_float(a4[c + 3]));
                    } else if (D != 64) {
                        __nv_bfloat16* dst = (half2 ? dk : dv) + orow + cb * 32;
#pragma unroll
                        for (int c = 0; c < 32; c += 8) {
                            uint32_t w4[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(a4[c + 2 * u]), __uint_as_float(a4[c + 2 * u + 1]));
                                w4[u] = *reinterpret_cast<uint32_t*>(&h);
                            }
                            *reinterpret_cast<uint4*>(dst + c) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                        }
                    }
                }
                if (D == 64 && !is_ret && !F32OUT) {
                    // window tile, bf16 out: the rows go into the (now idle) P^T / dS^T operand buffers in the swizzled
                    // layout and leave as one tile store per warp (a 128-byte store per thread stalls the load/store unit)
                    const uint32_t buf = half2 ? sDST : sPT;
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        uint32_t w4[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(a4[g * 8 + 2 * u]), __uint_as_float(a4[g * 8 + 2 * u + 1]));
                            w4[u] = *reinterpret_cast<uint32_t*>(&h);
                        }
                        const int ch = cb * 4 + g;
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(buf + tid * 128 + ((ch ^ (tid & 7)) << 4)),
                                     "r"(w4[0]), "r"(w4[1]), "r"(w4[2]), "r"(w4[3]) : "memory");
                    }
                }
            }
        }
        if (D == 64 && !is_ret && !F32OUT) {
            fence_proxy_async();
            __syncwarp();
            if (lane == 0 && j0 + warp * 32 < Tlen) {
                tma_store_3d(&tmDV, sPT + warp * 4096, 0, j0 + warp * 32, bh);
                tma_store_3d(&tmDK, sDST + warp * 4096, 0, j0 + warp * 32, bh);
                bulk_commit();
                bulk_wait_read0();                             // the buffers are released with the CTA
            }
        }
        if (live) {
            if (is_ret) dr_ret[(size_t)bh * R + e0 + tid] = dr;
            else dr_win[(size_t)bh * Tlen + pos] = dr;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, S::TMEM_COLS);
}

// Far-query share of the retained keys added onto their rows (each key appears once in the list: fixed order).
template <bool F32OUT>
__global__ void bwd_merge_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ cnt,
                                 const float* __restrict__ dk_ret, const float* __restrict__ dv_ret,
                                 const float* __restrict__ dr_ret, __nv_bfloat16* __restrict__ dk,
                                 __nv_bfloat16* __restrict__ dv, float* __restrict__ dk32, float* __restrict__ dv32,
                                 float* __restrict__ dr_win, int Tlen, int R, int D)
{
    pdl_launch_dependents();
    pdl_wait();                                                // see launch_pdl: earlier kernels of the stream have completed
    const int bh = blockIdx.y, e = blockIdx.x;
    if (e >= cnt[bh]) return;
    const int j = idx[(size_t)bh * R + e];
    const size_t src = ((size_t)bh * R + e) * D, dst = ((size_t)bh * Tlen + j) * D;
    for (int c = threadIdx.x; c < D; c += blockDim.x) {
        if (F32OUT) { dk32[dst + c] += dk_ret[src + c]; dv32[dst + c] += dv_ret[src + c]; }
        else {
            dk[dst + c] = __float2bfloat16_rn(__bfloat162float(dk[dst + c]) + dk_ret[src + c]);
            dv[dst + c] = __float2bfloat16_rn(__bfloat162float(dv[dst + c]) + dv_ret[src + c]);
        }
    }
    if (threadIdx.x == 0) dr_win[(size_t)bh * Tlen + j] += dr_ret[(size_t)bh * R + e];
}

// dr -> dz in place: Eq. 6 (+ Eq. 7's lambda term) through the sigmoid, for scored tokens only.
__global__ void bwd_dz_kernel(float* __restrict__ dz, const float* __restrict__ z, const float* __restrict__ lambda, int H,
                              int Tlen, int half, float zthr)
{
    pdl_launch_dependents();
    pdl_wait();                                                // see launch_pdl: earlier kernels of the stream have completed
    const int bh = blockIdx.y;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= Tlen) return;
    float g = 0.f;
    if (j + half <= Tlen - 1) {
        const float zz = z[(size_t)bh * Tlen + j];
        const float r = 1.f / (1.f + expf(-zz));
        float dr = dz[(size_t)bh * Tlen + j];
        if (lambda && zz > zthr) dr += lambda[bh % H];
        g = dr * r * (1.f - r);
    }
    dz[(size_t)bh * Tlen + j] = g;
}

}  // namespace

// dq (and delta) on the tensor cores.  Returns LTE_OK or an error; the caller runs the remaining stages.
int launch_bwd_dq_tc(const Params& p, const void* q, const void* k, const void* v, const void* o, const float* lse,
                     const void* dO, const int32_t* idx, const int32_t* cnt, void* dq, float* delta, cudaStream_t st)
{
    const int BHK = p.B * p.H, BH = BHK * p.G;                 // key/value heads, query heads
    CUtensorMap tq, tdo, to, tdq, tk, tv;
    if (!make_map(&tq, q, BH, p.T, p.d, BM) || !make_map(&tdo, dO, BH, p.T, p.d, BM) || !make_map(&to, o, BH, p.T, p.d, BM) ||
        !make_map(&tdq, dq, BH, p.T, p.d, 32) ||
        !make_map(&tk, k, BHK, p.T, p.d, BN) || !make_map(&tv, v, BHK, p.T, p.d, BN))
        return LTE_ERR_CUDA;
    dim3 grid((p.T + BM - 1) / BM, BH);
#define LTE_GO(D)                                                                                                  \
    do {                                                                                                           \
        static PerDeviceOnce attr;                                                                                 \
        if (int e = attr.run([] { return cudaFuncSetAttribute(bwd_dq_tc_kernel<D>,                                 \
                cudaFuncAttributeMaxDynamicSharedMemorySize, SmemQ<D>::BYTES); })) return e;                       \
        launch_pdl(bwd_dq_tc_kernel<D>, grid, dim3(NTHREADS), SmemQ<D>::BYTES, st,                            \
            tq, tdo, to, tdq, tk, tv, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)o,        \
            (const __nv_bfloat16*)dO, lse, idx, cnt, (__nv_bfloat16*)dq, delta, p.T, p.W, p.R, p.scale, p.G, p.d); \
    } while (0)
    if (p.d == 64 || p.d == 32) LTE_GO(64); else if (p.d == 128) LTE_GO(128); else return LTE_ERR_UNSUPPORTED;
#undef LTE_GO
    return cuda_status(cudaGetLastError());
}

// dk, dv, dz on the tensor cores.  `ret_ws` holds dk_ret, dv_ret [B,H,R,d] and dr_ret [B,H,R] (fp32).
size_t bwd_tc_ret_bytes(const Params& p)
{
    const size_t n = (size_t)p.B * p.H * (p.R > 0 ? p.R : 1);
    return ((2 * n * p.d + n) * 4 + 255) / 256 * 256;
}

int launch_bwd_dkv_tc(const Params& p, const void* q, const void* k, const void* v, const float* lse, const void* dO,
                      const float* delta, const float* z, const int32_t* idx, const int32_t* cnt, const float* lambda,
                      void* dk, void* dv, float* dk32, float* dv32, float* dz, void* ret_ws, bool f32out, bool merge_here,
                      cudaStream_t st)
{
    const int BH = p.B * p.H;
    CUtensorMap tk, tv, tq, tdo, tdk, tdv;
    if (!make_map(&tk, k, BH, p.T, p.d, 128) || !make_map(&tv, v, BH, p.T, p.d, 128) ||
        !make_map(&tq, q, BH * p.G, p.T, p.d, 64) || !make_map(&tdo, dO, BH * p.G, p.T, p.d, 64) ||
        !make_map(&tdk, dk, BH, p.T, p.d, 32) || !make_map(&tdv, dv, BH, p.T, p.d, 32))
        return LTE_ERR_CUDA;
    const size_t n = (size_t)BH * (p.R > 0 ? p.R : 1);
    float* dk_ret = (float*)ret_ws;
    float* dv_ret = dk_ret + n * p.d;
    float* dr_ret = dv_ret + n * p.d;
    const int n_wt = (p.T + 127) / 128, n_rt = (p.R + 127) / 128;
    dim3 grid(n_wt + n_rt, BH);
#define LTE_GO(D, F)                                                                                               \
    do {                                                                                                           \
        static PerDeviceOnce attr;                                                                                 \
        if (int e = attr.run([] { return cudaFuncSetAttribute(bwd_dkv_tc_kernel<D, F>,                             \
                cudaFuncAttributeMaxDynamicSharedMemorySize, SmemK<D>::BYTES); })) return e;                       \
        launch_pdl(bwd_dkv_tc_kernel<D, F>, grid, dim3(NTHREADS), SmemK<D>::BYTES, st,                              \
            tk, tv, tq, tdo, tdk, tdv, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, lse, delta, idx, cnt,     \
            (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, dk32, dv32, dz, dk_ret, dv_ret, dr_ret, n_wt, p.T, p.W, p.R,   \
            p.scale, p.G, p.d);                                                                                    \
    } while (0)
    if (p.d == 64 || p.d == 32) { if (f32out) LTE_GO(64, true); else LTE_GO(64, false); }
    else if (p.d == 128) { if (f32out) LTE_GO(128, true); else LTE_GO(128, false); }
    else return LTE_ERR_UNSUPPORTED;
#undef LTE_GO
    // merge_here = false: the caller's last pass adds the retained shares and turns dr into dz itself
    if (!merge_here) return cuda_status(cudaGetLastError());
    if (p.R > 0) {
        dim3 gm(p.R, BH);
        if (f32out)
            launch_pdl(bwd_merge_kernel<true>, gm, dim3(64), 0, st, idx, cnt, dk_ret, dv_ret, dr_ret, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv,
                                                      dk32, dv32, dz, p.T, p.R, p.d);
        else
            launch_pdl(bwd_merge_kernel<false>, gm, dim3(64), 0, st, idx, cnt, dk_ret, dv_ret, dr_ret, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv,
                                                       dk32, dv32, dz, p.T, p.R, p.d);
    }
    dim3 gz((p.T + 255) / 256, BH);
    launch_pdl(bwd_dz_kernel, gz, dim3(256), 0, st, dz, z, lambda, p.H, p.T, p.half, p.zthr);
    return cuda_status(cudaGetLastError());
}

int bwd_status_fetch_and_clear() { return status_fetch_and_clear(g_bwd_status); }

}  // namespace lte
