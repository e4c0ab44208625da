// Prefill attention on the 5th-generation tensor cores (Section 3.1.3, "Cached prefilling and decoding").
//
// One CTA per 128-query tile of one (b,h): four softmax warps and one control warp.  Key/value tiles of 64
// rows come from two sources, as in the paper's two-stage loop: (1) the contiguous window span, staged by TMA
// (cp.async.bulk.tensor, 128-byte swizzle); (2) the retained rows already out of the tile's window, gathered
// row by row with cp.async into the same swizzled layout (idx is ascending, so the entries a query may see are
// a prefix of the list and every mask is a column range).  Per tile:
//   S = Q K^T      tcgen05.mma (kind::f16, bf16 in, fp32 out) into one of two TMEM buffers, so the next two
//                  S tiles are computed while the softmax of the current one runs
//   softmax        thread r owns query row r = TMEM lane r: tcgen05.ld, range mask (whole 32-column chunks are
//                  skipped or taken unmasked when the warp's rows allow it), running max / sum in fp32 (exp2 with
//                  the scale folded in), P written as bf16 back into TMEM over the S buffer it came from
//   O += P V       tcgen05.mma with P as the TMEM A operand and V as an MN-major shared-memory operand,
//                  accumulated in TMEM; the accumulator is rescaled
//                  in place only when a row's maximum grows by more than 2^8 (lazy rescale)
// Loads run two to three tiles ahead of the tensor core.  Every mbarrier wait is bounded; a wait that runs out
// records a status word and the kernel still terminates.
#include "tc_common.cuh"

namespace lte {

__device__ int g_prefill_status = 0;          // 0 = fine; otherwise the code of the wait that gave up

#ifdef LTE_PROFILE
__device__ long long g_prof[160];
#define PROFC(slot) do { if (blockIdx.x == 5 && blockIdx.y == 3 && threadIdx.x == 128 && (slot) < 160) g_prof[slot] = clock64(); } while (0)
#define PROF(slot) do { if (blockIdx.x == 5 && blockIdx.y == 3 && threadIdx.x == 64) g_prof[slot] = clock64(); } while (0)
#else
#define PROF(slot) do { } while (0)
#define PROFC(slot) do { } while (0)
#endif

namespace {

constexpr int BM = 128, BN = 64, NTHREADS = 160;
using namespace tc;
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, int code) { mbar_wait_s(bar, parity, code, &g_prefill_status); }

template <int D> struct Smem {
    static constexpr int SUB = D / 64;                        // 64-column (128-byte) sub-tiles per row
    static constexpr int KST = 3;                             // key stages
    static constexpr int VST = D == 64 ? 3 : 2;               // value stages
    static constexpr int QTILE = BM * D * 2;                  // [128][D] bf16
    static constexpr int KVTILE = BN * D * 2;                 // [64][D] bf16
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = QTILE;
    static constexpr int OFF_V = OFF_K + KST * KVTILE;
    static constexpr int OFF_P = OFF_V + VST * KVTILE;        // (P lives in TMEM; nothing here)
    // d = 64: the row sums are taken by the tensor core as well: PV gets 16 extra B columns of ones, so column D of
    // the accumulator is sum_j P_ij of exactly the (bf16-rounded) probabilities the product used.  The ones live in one
    // more 64-column group, LBO away from the value tile.
    static constexpr bool ONES = D == 64;
    static constexpr int OFF_ONES = OFF_P;                    // [64][64] bf16 ones (8 KB), d = 64 only
    static constexpr int OFF_BAR = OFF_ONES + (ONES ? BN * 128 : 0);   // mbarriers, tmem slot
    static constexpr int OFF_IDX = OFF_BAR + 128;             // 128 staged list entries
    static constexpr int BYTES = OFF_IDX + 512;
    static constexpr uint32_t TMEM_COLS = 256;                // S0: [0,64)  S1: [64,128)  O: [128, 128+D) (+16 row-sum columns)
};

__device__ __forceinline__ void softmax_group_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Warps 0-3 (128 threads): softmax (thread r owns query row r) and the cp.async gathers of retained rows.
// Warp 4, one lane: the TMA loads of Q and of the window tiles, and every tcgen05.mma.  They meet on mbarriers:
//   bar_s[b]  (commit)       S(t) is in TMEM buffer b = t & 1                     control -> softmax
//   bar_p     (128 arrivals) P(t) is in shared memory, S buffer b is free         softmax -> control
//   bar_pv    (commit)       PV(t) has completed                                   control -> softmax
//   bar_g[b]  (128 arrivals) gathers issued before the top of tile t have landed   softmax -> control
//   bar_k[s], bar_v[s]       TMA transaction barriers of the window tiles
// S(t+1) and S(t+2) are computed while the softmax of tile t runs; loads run two to three tiles ahead.
template <int D>
__global__ void __launch_bounds__(NTHREADS, 2)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const __nv_bfloat16* __restrict__ kg,
                  const __nv_bfloat16* __restrict__ vg, const int32_t* __restrict__ idx,
                  const int32_t* __restrict__ cnt, __nv_bfloat16* __restrict__ o, float* __restrict__ lse, int Tlen,
                  int W, int R, float scale)
{
    using S = Smem<D>;
    constexpr int SUB = S::SUB, KST = S::KST, VST = S::VST;
    constexpr uint32_t TMEM_COLS = S::TMEM_COLS;
    constexpr uint32_t O_COL = 2 * BN;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 1023u) != 0) {                                 // the swizzled tiles need 1024-byte alignment
        if (threadIdx.x == 0) atomicExch(&g_prefill_status, 9);
        return;
    }
    PROF(0);
    const uint32_t sQ = base + S::OFF_Q, sK = base + S::OFF_K, sV = base + S::OFF_V;
    const uint32_t bar_q = base + S::OFF_BAR;
    const uint32_t bar_k0 = bar_q + 8;                         // 3 slots
    const uint32_t bar_v0 = bar_q + 32;                        // 3 slots
    const uint32_t bar_s0 = bar_q + 56;                        // 2 slots
    const uint32_t bar_g0 = bar_q + 72;                        // 2 slots
    const uint32_t bar_p = bar_q + 88, bar_pv = bar_q + 96;
    const uint32_t tmem_slot = bar_q + 104;
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_raw + S::OFF_BAR + 104);
    volatile int* s_idx = reinterpret_cast<volatile int*>(smem_raw + S::OFF_IDX);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.y;
    const int i0 = blockIdx.x * BM;
    const int i_hi = min(i0 + BM - 1, Tlen - 1);
    const int j_start = max(i0 - W + 1, 0);
    const int n_win = (i_hi - j_start + 1 + BN - 1) / BN;
    const int32_t* id = idx + (size_t)bh * R;
    const int n_ret = cnt[bh];

    if (tid == 0) {
        mbar_init(bar_q, 1);
#pragma unroll
        for (int s2 = 0; s2 < 3; ++s2) { mbar_init(bar_k0 + 8 * s2, 1); mbar_init(bar_v0 + 8 * s2, 1); }
        mbar_init(bar_s0, 1); mbar_init(bar_s0 + 8, 1);
        mbar_init(bar_g0, 128); mbar_init(bar_g0 + 8, 128);
        mbar_init(bar_p, 128); mbar_init(bar_pv, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;
    PROF(1);

    if (warp == 4) {
        // =================================== control warp (one lane) ========================================
        // number of tiles: retained entries visible to the last row of the tile (idx ascending => a prefix)
        int nv_max = 0;
        {
            const int lim = i_hi - W;
            for (int e0 = 0; e0 < n_ret; e0 += 32) {
                const int e = e0 + lane < n_ret ? id[e0 + lane] : 0x7fffffff;
                const unsigned bal = __ballot_sync(0xffffffffu, e <= lim);
                nv_max += __popc(bal);
                if (bal != 0xffffffffu) break;
            }
        }
        const int n_tiles = n_win + (nv_max + BN - 1) / BN;
        if (lane == 0) {
            constexpr uint32_t IDESC_S = instr_desc(BM, BN, false);
            constexpr uint32_t IDESC_O = S::ONES ? instr_desc(BM, D + 16, true) : instr_desc(BM, D, true);
            // descriptor words: lo = (address >> 4) | LBO field, hi = SBO field | version | swizzle mode
            constexpr uint32_t HI = (1024u >> 4) | (1u << 14) | (2u << 29);
            const uint32_t q_lo = (sQ >> 4) | (1u << 16), k_lo = (sK >> 4) | (1u << 16);
            const uint32_t v_lo = (sV >> 4) | ((8192u >> 4) << 16);
            uint32_t k_phase = 0, v_phase = 0, g_waited = 0;   // TMA barrier parities (bit per stage); bar_g phases consumed
            auto tma_kv = [&](int t, bool is_v) {              // window tile t -> its stage
                const int st = is_v ? (t % VST) : (t % KST);
                const uint32_t dst = (is_v ? sV : sK) + st * S::KVTILE;
                const uint32_t bar = (is_v ? bar_v0 : bar_k0) + 8 * st;
                mbar_expect_tx(bar, S::KVTILE);
                const int y = j_start + t * BN;
#pragma unroll
                for (int sb = 0; sb < SUB; ++sb) tma_load_3d(dst + sb * 8192, is_v ? &tmV : &tmK, sb * 64, y, bh, bar);
            };
            auto need_g = [&](uint32_t phase) {                // gathers issued before the top of tile `phase` have landed
                while (g_waited <= phase) { mbar_wait(bar_g0 + 8 * (g_waited & 1), (g_waited >> 1) & 1, 10); ++g_waited; }
            };
            auto wait_k = [&](int t) {
                if (t < n_win) { const int st = t % KST; mbar_wait(bar_k0 + 8 * st, (k_phase >> st) & 1u, 2); k_phase ^= 1u << st; }
            };
            auto wait_v = [&](int t) {
                if (t < n_win) { const int st = t % VST; mbar_wait(bar_v0 + 8 * st, (v_phase >> st) & 1u, 4); v_phase ^= 1u << st; }
            };
            auto mma_s = [&](int t) {
                const uint32_t kb = k_lo + (uint32_t)(t % KST) * (S::KVTILE >> 4);
                const uint32_t dcol = tmem + (t & 1) * BN;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                    umma(dcol, desc64(q_lo + (kk >> 2) * 1024 + (kk & 3) * 2, HI), desc64(kb + (kk >> 2) * 512 + (kk & 3) * 2, HI),
                         IDESC_S, kk > 0);
                umma_commit(bar_s0 + 8 * (t & 1));
            };

            mbar_expect_tx(bar_q, S::QTILE);
#pragma unroll
            for (int sb = 0; sb < SUB; ++sb) tma_load_3d(sQ + sb * 16384, &tmQ, sb * 64, i0, bh, bar_q);
            for (int t = 0; t < KST && t < n_win; ++t) tma_kv(t, false);
            for (int t = 0; t < VST && t < n_win; ++t) tma_kv(t, true);

            need_g(0);                                         // the softmax warps' prologue gathers
            mbar_wait(bar_q, 0, 1);
            wait_k(0);
            tc_fence_after();
            mma_s(0);
            if (n_tiles > 1) { wait_k(1); mma_s(1); }
            // K(KST) reuses the stage of K(0): S(0) must have completed
            if (KST < n_win) { mbar_wait(bar_s0, 0, 6); tma_kv(KST, false); }

            for (int t = 0; t < n_tiles; ++t) {
                // A. PV(t)
                need_g(t);
                mbar_wait(bar_p, t & 1, 7);
                wait_v(t);
                tc_fence_after();
                {
                    uint32_t vb = v_lo + (uint32_t)(t % VST) * (S::KVTILE >> 4);
                    if (S::ONES)   // second 64-column group of B = the block of ones: LBO = its distance from this value tile
                        vb = ((sV + (t % VST) * S::KVTILE) >> 4) | (((base + S::OFF_ONES - sV - (t % VST) * S::KVTILE) >> 4) << 16);
#pragma unroll
                    for (int kk = 0; kk < BN / 16; ++kk)
                        umma_ts(tmem + O_COL, tmem + (t & 1) * BN + kk * 8, desc64(vb + kk * 128, HI), IDESC_O, (t > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(bar_pv);
                }
                // B. S(t+2) into the S buffer softmax(t) has just released
                if (t + 2 < n_tiles) {
                    if (KST == 2) need_g(t + 1);
                    wait_k(t + 2);
                    mma_s(t + 2);
                }
                // C. window K(t+1+KST) reuses the stage of K(t+1): S(t+1) must have completed
                if (t + 1 + KST < n_win) {
                    mbar_wait(bar_s0 + 8 * ((t + 1) & 1), ((t + 1) >> 1) & 1, 6);
                    tma_kv(t + 1 + KST, false);
                }
                // D. window V(t-1+VST) reuses the stage of V(t-1); PV(t-1) is known to be complete because the
                //    softmax warps waited for it before they produced P(t)
                if (t >= 1 && t - 1 + VST < n_win) tma_kv(t - 1 + VST, true);
            }
        }
    } else {
        // =================================== softmax warps ==================================================
        const int i = i0 + tid;                                // this thread's query row
        // retained entries visible to this row: the list is staged through shared memory 128 entries at a time
        const int lim = min(i, Tlen - 1) - W;                  // entry visible iff idx <= lim
        const int lim_max = i_hi - W;
        int nvis = 0;
        for (int e0 = 0; e0 < n_ret; e0 += 128) {
            const int n_here = min(128, n_ret - e0);
            softmax_group_sync();
            if (tid < n_here) s_idx[tid] = id[e0 + tid];
            softmax_group_sync();
            if (s_idx[n_here - 1] <= lim) nvis += n_here;
            else {
                int lo = 0, hi = n_here;
                while (lo < hi) { const int mid = (lo + hi) >> 1; if (s_idx[mid] <= lim) lo = mid + 1; else hi = mid; }
                nvis += lo;
            }
            if (s_idx[n_here - 1] > lim_max) break;            // uniform: nothing further is visible to any row
        }
        softmax_group_sync();                                  // every search in the staging buffer is done
        if (i == i_hi) s_idx[0] = nvis;                        // the tile count follows the last valid row
        softmax_group_sync();
        const int nv_max = s_idx[0];
        const int n_tiles = n_win + (nv_max + BN - 1) / BN;
        PROF(2);

        // gather of one retained tile: 8 lanes per row copy its 16-byte chunks (coalesced reads, conflict-free
        // swizzled writes), 16 rows per pass; rows past the visible prefix are zero-filled
        const int g_row = tid >> 3, g_sub = tid & 7;
        auto gather_rows = [&](int t, int (&rows4)[4]) {       // row positions of this thread's 4 rows of tile t
#pragma unroll
            for (int ps = 0; ps < 4; ++ps) {
                const int e = (t - n_win) * BN + ps * 16 + g_row;
                rows4[ps] = (t >= n_win && t < n_tiles && e < nv_max) ? id[e] : -1;
            }
        };
        auto gather_issue = [&](int t, bool is_v, const int (&rows4)[4]) {
            if (t >= n_win && t < n_tiles) {
                const int st = is_v ? (t % VST) : (t % KST);
                const uint32_t dst = (is_v ? sV : sK) + st * S::KVTILE;
#pragma unroll
                for (int ps = 0; ps < 4; ++ps) {
                    const int row = ps * 16 + g_row;
                    const bool ok = rows4[ps] >= 0;
                    const __nv_bfloat16* src = (is_v ? vg : kg) + ((size_t)bh * Tlen + (ok ? rows4[ps] : 0)) * D;
#pragma unroll
                    for (int c = g_sub; c < D / 8; c += 8) {
                        const uint32_t off = (c >> 3) * 8192 + row * 128 + (((c & 7) ^ (row & 7)) << 4);
                        cp_async16(dst + off, src + c * 8, ok ? 16u : 0u);
                    }
                }
            }
            cp_async_commit();
        };
        // prologue gathers: the first KST key tiles and VST value tiles (those that are retained tiles)
        {
            int rows4[4];
            for (int t = 0; t < KST; ++t) { gather_rows(t, rows4); gather_issue(t, false, rows4); }
            for (int t = 0; t < VST; ++t) { gather_rows(t, rows4); gather_issue(t, true, rows4); }
        }

        if (S::ONES) {                                         // 8 KB of bf16 1.0: 64 bytes per thread
#pragma unroll
            for (int u = 0; u < 4; ++u)
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base + S::OFF_ONES + tid * 64 + u * 16), "r"(0x3F803F80u) : "memory");
        }
        const float c2 = scale * 1.4426950408889634f;          // logits are handled in the log2 domain: x = s * c2
        const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;   // this warp's TMEM lanes
        float m_run = -INFINITY, l_run = 0.f;                  // running max (log2 domain) and sum (sum only if !ONES)

        for (int t = 0; t < n_tiles; ++t) {
            // row positions for this tile's two gathers, fetched first so their latency hides under the softmax
            int rk[4], rv[4];
            gather_rows(t + KST, rk);
            gather_rows(t + VST - 1, rv);
            // gathers issued before this point have landed (all of them, or all but the latest value tile)
            if (VST == 3) cp_async_wait<1>(); else cp_async_wait<0>();
            fence_proxy_async();
            mbar_arrive(bar_g0 + 8 * (t & 1));

            // column range this row may see in the tile
            int c_lo, c_hi;
            if (t < n_win) {
                const int jt0 = j_start + t * BN;
                c_lo = max(i - W + 1, 0) - jt0;
                c_hi = i - jt0;
            } else {
                c_lo = 0;
                c_hi = nvis - (t - n_win) * BN - 1;
            }
            // rows of a warp are consecutive and both bounds grow with the row: lane 0 / lane 31 give the warp's
            // union range (columns any row sees) and intersection range (columns every row sees)
            const int u_lo = __shfl_sync(0xffffffffu, c_lo, 0), u_hi = __shfl_sync(0xffffffffu, c_hi, 31);
            const int n_lo = __shfl_sync(0xffffffffu, c_lo, 31), n_hi = __shfl_sync(0xffffffffu, c_hi, 0);
            bool act[2], full[2];
            uint32_t vm[2];                                    // per-thread validity bits of a partial chunk
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                const int lo = cb * 32, hi = lo + 31;
                act[cb] = lo <= u_hi && hi >= u_lo;
                full[cb] = lo >= n_lo && hi <= n_hi;
                const int a = min(max(c_lo - lo, 0), 32), b2 = min(max(c_hi - lo + 1, 0), 32);
                const uint32_t below_b = b2 >= 32 ? 0xffffffffu : ((1u << b2) - 1u);
                const uint32_t below_a = a >= 32 ? 0xffffffffu : ((1u << a) - 1u);
                vm[cb] = b2 > a ? (below_b & ~below_a) : 0u;
            }

            PROF(4 + 6 * t);
            mbar_wait(bar_s0 + 8 * (t & 1), (t >> 1) & 1, 3);  // S(t) is in TMEM buffer t & 1
            tc_fence_after();
            PROF(5 + 6 * t);
            gather_issue(t + KST, false, rk);                  // its stage held K(t), which S(t) has finished reading
            const uint32_t s_col = (t & 1) * BN;
            uint32_t r[2][32];
#pragma unroll
            for (int cb = 0; cb < 2; ++cb)
                if (act[cb]) tmem_ld32(tmem + lane_base + s_col + cb * 32, r[cb]);
            tmem_wait_ld();
            PROF(6 + 6 * t);
            float mr[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // row max of the raw logits, 4 chains
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                if (!act[cb]) continue;
                if (full[cb]) {
#pragma unroll
                    for (int c = 0; c < 32; c += 2)
                        mr[(c >> 1) & 3] = max3(mr[(c >> 1) & 3], __uint_as_float(r[cb][c]), __uint_as_float(r[cb][c + 1]));
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const float x = (vm[cb] & (1u << c)) ? __uint_as_float(r[cb][c]) : -INFINITY;
                        r[cb][c] = __float_as_uint(x);
                        mr[c & 3] = fmaxf(mr[c & 3], x);
                    }
                }
            }
            const float m_tile = fmaxf(fmaxf(mr[0], mr[1]), fmaxf(mr[2], mr[3])) * c2;
            PROF(7 + 6 * t);
            // PV(t-1) must be done before O is rescaled or P is overwritten
            if (t > 0) { mbar_wait(bar_pv, (t - 1) & 1, 4); tc_fence_after(); }
            PROF(8 + 6 * t);
            // value tile t+VST-1 goes into the stage of V(t-1), which PV(t-1) has finished reading
            if (t > 0) gather_issue(t + VST - 1, true, rv); else cp_async_commit();
            // lazy rescale: the running max only moves when the new one is far above it (exp2 arguments stay <= 8)
            float alpha = 1.f;
            bool need = false;
            if (m_run == -INFINITY) m_run = m_tile;             // nothing accumulated yet for this row: O row is 0
            else if (m_tile > m_run + 8.f) { alpha = fast_exp2(m_run - m_tile); m_run = m_tile; need = true; }
            if (__any_sync(0xffffffffu, need)) {
#pragma unroll
                for (int cb = 0; cb < D / 32 + (S::ONES ? 1 : 0); ++cb) {   // with ONES the row-sum columns are rescaled too
                    uint32_t q4[32];
                    tmem_ld32(tmem + lane_base + O_COL + cb * 32, q4);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; ++c) q4[c] = __float_as_uint(__uint_as_float(q4[c]) * alpha);
                    tmem_st32(tmem + lane_base + O_COL + cb * 32, q4);
                }
                tmem_wait_st();
                l_run *= alpha;
            }
            const float neg_m = m_run == -INFINITY ? 0.f : -m_run;
            float ls[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t pk[32];                                   // the row of P as 64 bf16, two per word
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                if (act[cb]) {
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        // masked entries hold -inf: fma gives -inf and exp2(-inf) = 0
                        const float p0 = fast_exp2(fmaf(__uint_as_float(r[cb][c]), c2, neg_m));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(r[cb][c + 1]), c2, neg_m));
                        if (!S::ONES) ls[(c >> 1) & 3] += p0 + p1;   // with ONES the tensor core sums the rounded probabilities
                        __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                        pk[cb * 16 + (c >> 1)] = *reinterpret_cast<uint32_t*>(&h);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 16; ++c) pk[cb * 16 + c] = 0u;
                }
            }
            l_run += (ls[0] + ls[1]) + (ls[2] + ls[3]);
            // P goes back into TMEM, over the first 32 columns of the S buffer it was computed from (this thread has
            // all of its row in registers), and feeds the PV product as the A operand: no trip through shared memory
            tmem_st32(tmem + lane_base + s_col, pk);
            tmem_wait_st();
            tc_fence_before();                                 // our TMEM accesses are ordered before the arrive
            mbar_arrive(bar_p);
            PROF(9 + 6 * t);
        }
        PROF(50);
        mbar_wait(bar_pv, (n_tiles - 1) & 1, 5);
        tc_fence_after();
        PROF(51);

        // ---- epilogue: O / l -> bf16, logsumexp ----------------------------------------------------------
        if (S::ONES) {                                         // the row sum is column D of the accumulator
            uint32_t q4[32];
            tmem_ld32(tmem + lane_base + O_COL + D, q4);
            tmem_wait_ld();
            l_run = __uint_as_float(q4[0]);
        }
        const float inv = 1.f / l_run;
        __nv_bfloat16* orow = o + ((size_t)bh * Tlen + i) * D;
#pragma unroll
        for (int cb = 0; cb < D / 32; ++cb) {
            uint32_t q4[32];
            tmem_ld32(tmem + lane_base + O_COL + cb * 32, q4);
            tmem_wait_ld();
            if (i < Tlen) {
#pragma unroll
                for (int c = 0; c < 32; c += 8) {
                    uint32_t w4[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(q4[c + 2 * u]) * inv,
                                                                 __uint_as_float(q4[c + 2 * u + 1]) * inv);
                        w4[u] = *reinterpret_cast<uint32_t*>(&h);
                    }
                    *reinterpret_cast<uint4*>(orow + cb * 32 + c) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                }
            }
        }
        if (i < Tlen) lse[(size_t)bh * Tlen + i] = m_run * 0.6931471805599453f + logf(l_run);
        PROF(52);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, TMEM_COLS);
}

template <int D>
int run(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx, const int32_t* cnt, void* o,
        float* lse, cudaStream_t st)
{
    CUtensorMap tq, tk, tv;
    const int BH = p.B * p.H;
    if (!make_map(&tq, q, BH, p.T, D, BM) || !make_map(&tk, k, BH, p.T, D, BN) || !make_map(&tv, v, BH, p.T, D, BN))
        return LTE_ERR_CUDA;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(prefill_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::BYTES) !=
            cudaSuccess)
            return LTE_ERR_CUDA;
        attr_done = true;
    }
    dim3 grid((p.T + BM - 1) / BM, BH);
    prefill_tc_kernel<D><<<grid, NTHREADS, Smem<D>::BYTES, st>>>(tq, tk, tv, (const __nv_bfloat16*)k,
                                                                 (const __nv_bfloat16*)v, idx, cnt, (__nv_bfloat16*)o,
                                                                 lse, p.T, p.W, p.R, p.scale);
    return cuda_status(cudaGetLastError());
}

}  // namespace

int launch_prefill_tc(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx,
                      const int32_t* cnt, void* o, float* lse, cudaStream_t st)
{
    switch (p.d) {
        case 64: return run<64>(p, q, k, v, idx, cnt, o, lse, st);
        case 128: return run<128>(p, q, k, v, idx, cnt, o, lse, st);
    }
    return launch_prefill_simt(p, q, k, v, idx, cnt, o, lse, st);   // d = 32: rows too narrow for the 128-byte swizzle
}

#ifdef LTE_PROFILE
extern "C" int lte_prof_read(long long* out) { return cudaMemcpyFromSymbol(out, g_prof, sizeof(long long) * 160) == cudaSuccess ? 0 : -1; }
#endif

int prefill_status_fetch_and_clear()
{
    int h = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&h, g_prefill_status, sizeof(int)) != cudaSuccess) return -1;
    if (h != 0) cudaMemcpyToSymbol(g_prefill_status, &zero, sizeof(int));
    return h;
}

}  // namespace lte
