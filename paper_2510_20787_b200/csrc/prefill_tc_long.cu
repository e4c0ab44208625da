// Prefill attention on the 5th-generation tensor cores (Section 3.1.3), variant for long items: one CTA per
// 128-query tile of one (b,h), used at d = 128, where a tile walks ten and more key tiles and the hardware's block
// scheduler balances the load better than a static persistent schedule (and the registers a persistent loop
// keeps alive are not free).  The tile loop is the one of the persistent kernel:
//   S = Q K^T      tcgen05.mma (kind::f16, bf16 in, fp32 out) into one of two TMEM buffers
//   softmax        thread r owns query row r = TMEM lane r; P written as bf16 back into TMEM over its S buffer
//   O += P V       tcgen05.mma with P as the TMEM A operand and V as an MN-major shared-memory operand; lazy rescale
// Window tiles come by TMA, retained rows by cp.async gathers into the same swizzled layout.  Every mbarrier wait is
// bounded; a wait that runs out records a status word and the kernel still terminates.
#include "tc_common.cuh"

namespace lte {

__device__ StatusWord g_prefill_long_status = LTE_STATUS_INIT; // 0 = fine; otherwise the code of the wait that gave up


#ifdef LTE_PROFILE
// cycles per phase, summed over all CTAs: [0,16) softmax thread 0, [16,32) the MMA warp's lane 0
__device__ unsigned long long g_plprof[64];
// (accumulated in shared memory and flushed once per CTA: global atomics in the loop slowed the fences down)
#define PLM(k) do { if (prof_on) { const long long now_ = clock64(); prof_[(k) + pofs_] += (unsigned long long)(now_ - tprev_); tprev_ = now_; } } while (0)
#define PLM_INIT(cond) const bool prof_on = (cond); long long tprev_ = clock64(); int pofs_ = 0
#define PLM_TILE(t) pofs_ = (t) >= n_win ? 32 : 0
#define PLM_FLUSH(lo, hi) do { if (prof_on) for (int k_ = lo; k_ < hi; ++k_) { atomicAdd(&g_plprof[k_], prof_[k_]); atomicAdd(&g_plprof[k_ + 32], prof_[k_ + 32]); } } while (0)
#else
#define PLM(k) do { } while (0)
#define PLM_INIT(cond) do { } while (0)
#define PLM_TILE(t) do { } while (0)
#define PLM_FLUSH(lo, hi) do { } while (0)
#endif

namespace {

constexpr int BM = 128, BN = 64, NTHREADS = 192;
using namespace tc;
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, int code) { mbar_wait_s(bar, parity, code, &g_prefill_long_status); }

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
#ifdef LTE_PROFILE
    static constexpr int BYTES = OFF_BAR + 768;
#else
    static constexpr int BYTES = OFF_BAR + 256;
#endif
    static constexpr uint32_t TMEM_COLS = 256;                // S0: [0,64)  S1: [64,128)  O: [128, 128+D) (+16 row-sum columns)
};


// Warps 0-3 (128 threads): softmax (thread r owns query row r) and the cp.async gathers of retained rows.
// Warp 4, one lane: every tcgen05.mma.  Warp 5, one lane: the TMA loads of Q and of the window tiles (a single
// lane doing both was the bottleneck: its dependent instruction stream took longer per tile than the softmax).
// They meet on mbarriers:
//   bar_s[b]  (commit)       S(t) is in TMEM buffer b = t & 1                     control -> softmax
//   bar_p     (128 arrivals) P(t) is in shared memory, S buffer b is free         softmax -> control
//   bar_pv[b] (commit)       PV(t) has completed, b = t & 1 (a barrier per parity: a waiter can then never find it two
//                            phases ahead, so the softmax threads wait on it only where they need the product)   control -> softmax
//   bar_gk[s], bar_gv[s] (128 arrivals, by cp.async completion) a gathered tile is in stage s   softmax -> control
//   bar_k[s], bar_v[s]       TMA transaction barriers of the window tiles
//   bar_kf[s], bar_vf[s]     (commit) the MMA that read stage s has completed          MMA lane -> load lane
// S(t+1) and S(t+2) are computed while the softmax of tile t runs; loads run two to three tiles ahead.
// STREAM (with compact): the list is every entry retained at some query of a chunk and entry e is gone from query leave[e] on
// (the streaming reading of a chunk): retained tiles take one more mask, leave > query position.
template <int D, bool compact, bool STREAM>
__global__ void __launch_bounds__(NTHREADS, 2)
prefill_long_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                  const __grid_constant__ CUtensorMap tmKc, const __grid_constant__ CUtensorMap tmVc,
                  const __nv_bfloat16* __restrict__ kg,
                  const __nv_bfloat16* __restrict__ vg, const int32_t* __restrict__ idx,
                  const int32_t* __restrict__ cnt, const int32_t* __restrict__ leave, __nv_bfloat16* __restrict__ o,
                  float* __restrict__ lse, int Tlen, int W, int R, float scale, int G, int qoff)
{
    using S = Smem<D>;
    constexpr int SUB = S::SUB, KST = S::KST, VST = S::VST;
    constexpr uint32_t TMEM_COLS = S::TMEM_COLS;
    constexpr uint32_t O_COL = 2 * BN;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 1023u) != 0) {                                 // the swizzled tiles need 1024-byte alignment
        if (threadIdx.x == 0) atomicExch(&g_prefill_long_status.code, 9);
        return;
    }
    const uint32_t sQ = base + S::OFF_Q, sK = base + S::OFF_K, sV = base + S::OFF_V;
    const uint32_t bar_q = base + S::OFF_BAR;
    const uint32_t bar_k0 = bar_q + 8;                         // 3 slots
    const uint32_t bar_v0 = bar_q + 32;                        // 3 slots
    const uint32_t bar_s0 = bar_q + 56;                        // 2 slots
    const uint32_t bar_p0 = bar_q + 88, bar_p1 = bar_q + 216, bar_pv0 = bar_q + 96, bar_pv1 = bar_q + 208;   // per tile parity
    const uint32_t bar_kf0 = bar_q + 104;                      // 3 slots: K stage free
    const uint32_t bar_vf0 = bar_q + 128;                      // 3 slots: V stage free
    const uint32_t tmem_slot = bar_q + 152;
    const uint32_t bar_gk0 = bar_q + 160, bar_gv0 = bar_q + 184;   // 3 slots each: a gathered tile has landed in the stage
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_raw + S::OFF_BAR + 152);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef LTE_PROFILE
    volatile unsigned long long* prof_ = reinterpret_cast<volatile unsigned long long*>(smem_raw + S::OFF_BAR + 256);
    if (tid < 64) prof_[tid] = 0ull;
#endif
    const int bh = blockIdx.y, bhk = bh / G;                   // query head and its key/value head (the G query heads of one are adjacent)
    const int i0 = qoff + blockIdx.x * BM;                     // positions; the query tensors start at position qoff
    const int i_hi = min(i0 + BM - 1, Tlen - 1);
    const int j_start = max(i0 - W + 1, 0);
    const int n_win = (i_hi - j_start + 1 + BN - 1) / BN;
    const int32_t* id = idx + (size_t)bhk * R;

    if (tid == 0) {
        mbar_init(bar_q, 1);
#pragma unroll
        for (int s2 = 0; s2 < 3; ++s2) {
            mbar_init(bar_k0 + 8 * s2, 1); mbar_init(bar_v0 + 8 * s2, 1);
            mbar_init(bar_kf0 + 8 * s2, 1); mbar_init(bar_vf0 + 8 * s2, 1);
        }
        mbar_init(bar_s0, 1); mbar_init(bar_s0 + 8, 1);
        // every softmax thread arrives itself: one arrival per warp behind a __syncwarp() lengthened the hand-over of P
        // to the MMA warp and cost 3 % at d = 128, T = 32768
#pragma unroll
        for (int s2 = 0; s2 < 3; ++s2) { mbar_init(bar_gk0 + 8 * s2, 128); mbar_init(bar_gv0 + 8 * s2, 128); }
        mbar_init(bar_p0, 128); mbar_init(bar_p1, 128); mbar_init(bar_pv0, 1); mbar_init(bar_pv1, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;
    pdl_launch_dependents();
    pdl_wait();                                                // everything above ran beside the previous kernel's tail
    // Q and the first window tiles need nothing but the tile's coordinates: they are on their way before the list is looked at
    const int n_early = min(n_win, Smem<D>::VST);
    if (warp == 5 && lane == 0) {
        mbar_expect_tx(bar_q, S::QTILE);
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb) tma_load_3d(sQ + sb * 16384, &tmQ, sb * 64, i0 - qoff, bh, bar_q);
        for (int t = 0; t < n_early; ++t) {
            mbar_expect_tx(bar_k0 + 8 * t, S::KVTILE);
            mbar_expect_tx(bar_v0 + 8 * t, S::KVTILE);
#pragma unroll
            for (int sb = 0; sb < SUB; ++sb) {
                tma_load_3d(sK + t * S::KVTILE + sb * 8192, &tmK, sb * 64, j_start + t * BN, bhk, bar_k0 + 8 * t);
                tma_load_3d(sV + t * S::KVTILE + sb * 8192, &tmV, sb * 64, j_start + t * BN, bhk, bar_v0 + 8 * t);
            }
        }
    }
    __syncwarp();
    const int n_ret = cnt[bhk];

    if (warp >= 4) {
        // ============================ load lane (warp 5) and MMA lane (warp 4) ==============================
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
        if (warp == 5 && lane == 0) {
            // ---- load lane: Q, then the window tiles, each into its stage as soon as the MMA that read the
            //      stage's previous tile has completed (bar_kf / bar_vf, one phase per use of a stage)
            // compact = 1: the retained rows were copied into contiguous tensors [B*H][R][d] beforehand (tmKc, tmVc), so the
            // retained tiles are TMA boxes like the window tiles; otherwise the softmax warps gather them
            const int n_load = compact ? n_tiles : n_win;
            auto load_tile = [&](int t, bool is_v, int st) {
                const uint32_t dst = (is_v ? sV : sK) + st * S::KVTILE;
                const uint32_t bar = (is_v ? bar_v0 : bar_k0) + 8 * st;
                const CUtensorMap* tm = t < n_win ? (is_v ? &tmV : &tmK) : (is_v ? &tmVc : &tmKc);
                const int y = t < n_win ? j_start + t * BN : (t - n_win) * BN;
                mbar_expect_tx(bar, S::KVTILE);
#pragma unroll
                for (int sb = 0; sb < SUB; ++sb) tma_load_3d(dst + sb * 8192, tm, sb * 64, y, bhk, bar);
            };
            int ks = 0, vs = 0;                                // stage of the next K / V tile to load
            uint32_t kf_par = 0, vf_par = 0;                   // parity bit per stage of the "free" barriers
            int tk = n_early, tv = n_early;                    // next tile to load (the first ones are already on their way)
            for (; tk < KST && tk < n_load; ++tk) load_tile(tk, false, tk);
            for (; tv < VST && tv < n_load; ++tv) load_tile(tv, true, tv);
            while (tk < n_load || tv < n_load) {
                if (tk < n_load) {                             // K(tk) into the stage of K(tk - KST)
                    mbar_wait(bar_kf0 + 8 * ks, (kf_par >> ks) & 1u, 6);
                    kf_par ^= 1u << ks;
                    load_tile(tk, false, ks);
                    ++tk;
                    ks = ks + 1 == KST ? 0 : ks + 1;
                }
                if (tv < n_load) {                             // V(tv) into the stage of V(tv - VST)
                    mbar_wait(bar_vf0 + 8 * vs, (vf_par >> vs) & 1u, 8);
                    vf_par ^= 1u << vs;
                    load_tile(tv, true, vs);
                    ++tv;
                    vs = vs + 1 == VST ? 0 : vs + 1;
                }
            }
        } else if (warp == 4) {
            // ---- MMA warp: nothing but barrier waits and tcgen05 issue; stage indices and parities roll.  The whole warp
            //      walks the loop and waits; only the tcgen05 instructions are guarded by the lane test, so that addresses
            //      and descriptors are computed in convergent code (cheaper to issue than from a loop run by one lane).
            constexpr uint32_t IDESC_S = instr_desc(BM, BN, false);
            constexpr uint32_t IDESC_O = S::ONES ? instr_desc(BM, D + 16, true) : instr_desc(BM, D, true);
            // descriptor words: lo = (address >> 4) | LBO field, hi = SBO field | version | swizzle mode
            constexpr uint32_t HI = (1024u >> 4) | (1u << 14) | (2u << 29);
            const uint32_t q_lo = (sQ >> 4) | (1u << 16), k_lo = (sK >> 4) | (1u << 16);
            // value operand: the second 64-column group of B is the next sub-tile (d = 128) or the block of ones
            // (d = 64, LBO = its distance from the value stage)
            uint32_t v_desc[VST];
#pragma unroll
            for (int st = 0; st < VST; ++st) {
                const uint32_t va = sV + st * S::KVTILE;
                v_desc[st] = (va >> 4) | ((S::ONES ? ((base + S::OFF_ONES - va) >> 4) : (8192u >> 4)) << 16);
            }
            uint32_t k_par = 0, v_par = 0, gk_par = 0, gv_par = 0;   // barrier parities, a bit per stage (TMA tiles; gathered tiles)
            int ks = 0, vs = 0;                                // stage of the next S / PV operand
            int ts = 0;                                        // next S tile to issue
            auto mma_s = [&]() {                               // S(ts) from K stage ks into S buffer ts & 1
                if (ts < n_win || compact) { mbar_wait(bar_k0 + 8 * ks, (k_par >> ks) & 1u, 2); k_par ^= 1u << ks; }
                else {                                         // gathered rows: generic-proxy writes, made visible to the tensor core here
                    mbar_wait(bar_gk0 + 8 * ks, (gk_par >> ks) & 1u, 10); gk_par ^= 1u << ks;
                    fence_proxy_async();
                }
                tc_fence_after();
                const uint32_t kb = k_lo + (uint32_t)ks * (S::KVTILE >> 4);
                const uint32_t dcol = tmem + (ts & 1) * BN;
                if (lane == 0) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        umma(dcol, desc64(q_lo + (kk >> 2) * 1024 + (kk & 3) * 2, HI), desc64(kb + (kk >> 2) * 512 + (kk & 3) * 2, HI),
                             IDESC_S, kk > 0);
                    umma_commit(bar_s0 + 8 * (ts & 1));
                    umma_commit(bar_kf0 + 8 * ks);             // the K stage is free once S(ts) has completed
                }
                __syncwarp();
                ++ts;
                ks = ks + 1 == KST ? 0 : ks + 1;
            };

            PLM_INIT(lane == 0);
            mbar_wait(bar_q, 0, 1);
            PLM(16);
            mma_s();                                           // tile 0 is always a window tile
            if (n_tiles > 1) mma_s();
            for (int t = 0; t < n_tiles; ++t) {
                // PV(t): everything but P is normally there long before
                PLM(17);
                PLM_TILE(t);
                if (t < n_win || compact) { mbar_wait(bar_v0 + 8 * vs, (v_par >> vs) & 1u, 4); v_par ^= 1u << vs; }
                else { mbar_wait(bar_gv0 + 8 * vs, (gv_par >> vs) & 1u, 11); gv_par ^= 1u << vs; fence_proxy_async(); }
                PLM(18);
                uint32_t vb = v_desc[0];
#pragma unroll
                for (int st = 1; st < VST; ++st) vb = vs == st ? v_desc[st] : vb;
                mbar_wait((t & 1) ? bar_p1 : bar_p0, (t >> 1) & 1, 7);
                PLM(19);
                tc_fence_after();
                if (lane == 0) {
#pragma unroll
                    for (int kk = 0; kk < BN / 16; ++kk)
                        umma_ts(tmem + O_COL, tmem + (t & 1) * BN + kk * 8, desc64(vb + kk * 128, HI), IDESC_O, (t > 0 || kk > 0) ? 1u : 0u);
                    umma_commit((t & 1) ? bar_pv1 : bar_pv0);
                    umma_commit(bar_vf0 + 8 * vs);             // the V stage is free once PV(t) has completed
                }
                __syncwarp();
                vs = vs + 1 == VST ? 0 : vs + 1;
                PLM(20);
                // S(t+2) into the S buffer softmax(t) has just released
                if (ts < n_tiles) mma_s();
                PLM(21);
            }
            PLM_FLUSH(16, 22);
        }
    } else {
        // =================================== softmax warps ==================================================
        const int i = i0 + tid;                                // this thread's query row
        if (S::ONES) {                                         // 8 KB of bf16 1.0: 64 bytes per thread
#pragma unroll
            for (int u = 0; u < 4; ++u)
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base + S::OFF_ONES + tid * 64 + u * 16), "r"(0x3F803F80u) : "memory");
        }
        // retained entries visible to this row.  The rows of a warp are consecutive and the list is ascending, so
        // nvis(row) = #{idx <= lim of lane 0} + #{idx in (lim of lane 0, lim of this lane]}: a ballot count plus a
        // 31-bit map of the entries that fall between the warp's first and last limit.  No block barrier.
        const int lim = min(i, Tlen - 1) - W;                  // entry visible iff idx <= lim
        const int lim_max = i_hi - W;
        const int lim0 = __shfl_sync(0xffffffffu, lim, 0), lim31 = __shfl_sync(0xffffffffu, lim, 31);
        int nvis = 0, nv_max = 0;                              // nv_max: entries visible to the tile's last row
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
                if (__shfl_sync(0xffffffffu, e[3], 31) > lim_max) break;   // nothing further is visible to any row
            }
            nvis += __popc(bits & ((1u << (lim - lim0)) - 1u));
        }
        const int n_tiles = n_win + (nv_max + BN - 1) / BN;
        const int iw0 = i0 + warp * 32;                        // the warp's first row
        const int nvis0 = __shfl_sync(0xffffffffu, nvis, 0), nvis31 = __shfl_sync(0xffffffffu, nvis, 31);

        // gather of one retained tile: 8 lanes per row copy its 16-byte chunks (coalesced reads, conflict-free
        // swizzled writes), 16 rows per pass; rows past the visible prefix are zero-filled
        const int g_row = tid >> 3, g_sub = tid & 7;
        auto gather_rows = [&](int t, int (&rows4)[4]) {       // row positions of this thread's 4 rows of tile t
#pragma unroll
            for (int ps = 0; ps < 4; ++ps) {
                const int e = (t - n_win) * BN + ps * 16 + g_row;
                rows4[ps] = (!compact && t >= n_win && t < n_tiles && e < nv_max) ? id[e] : -1;
            }
        };
        auto gather_issue = [&](int t, bool is_v, const int (&rows4)[4]) {
            if (!compact && t >= n_win && t < n_tiles) {
                const int st = is_v ? (t % VST) : (t % KST);
                const uint32_t dst = (is_v ? sV : sK) + st * S::KVTILE;
#pragma unroll
                for (int ps = 0; ps < 4; ++ps) {
                    const int row = ps * 16 + g_row;
                    const bool ok = rows4[ps] >= 0;
                    const __nv_bfloat16* src = (is_v ? vg : kg) + ((size_t)bhk * Tlen + (ok ? rows4[ps] : 0)) * D;
#pragma unroll
                    for (int c = g_sub; c < D / 8; c += 8) {
                        const uint32_t off = (c >> 3) * 8192 + row * 128 + (((c & 7) ^ (row & 7)) << 4);
                        cp_async16(dst + off, src + c * 8, ok ? 16u : 0u);
                    }
                }
                cp_async_arrive((is_v ? bar_gv0 : bar_gk0) + 8 * st);   // this thread's share of the tile has landed
            }
        };
        // prologue gathers: the first KST key tiles and VST value tiles (those that are retained tiles)
        if (n_win < KST) {
            int rows4[4];
            for (int t = 0; t < KST; ++t) { gather_rows(t, rows4); gather_issue(t, false, rows4); }
            for (int t = 0; t < VST; ++t) { gather_rows(t, rows4); gather_issue(t, true, rows4); }
        }

        const float c2 = scale * 1.4426950408889634f;          // logits are handled in the log2 domain: x = s * c2
        const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;   // this warp's TMEM lanes
        float m_run = -INFINITY, l_run = 0.f;                  // running max (log2 domain) and sum (sum only if !ONES)

        PLM_INIT(tid == 0);
        PLM(0);
        for (int t = 0; t < n_tiles; ++t) {
            PLM_TILE(t);
            // row positions for this tile's two gathers, fetched first so their latency hides under the softmax
            int rk[4], rv[4];
            gather_rows(t + KST, rk);
            gather_rows(t + VST - 1, rv);
            // column range this row may see in the tile
            // rows of a warp are consecutive and both bounds grow with the row: its first / last row give the warp's
            // union range (columns any row sees) and intersection range (columns every row sees)
            int c_lo, c_hi, u_lo, u_hi, n_lo, n_hi;
            if (t < n_win) {
                const int jt0 = j_start + t * BN;
                c_lo = max(i - W + 1, 0) - jt0;
                c_hi = i - jt0;
                u_lo = max(iw0 - W + 1, 0) - jt0; n_lo = max(iw0 + 31 - W + 1, 0) - jt0;
                n_hi = iw0 - jt0; u_hi = iw0 + 31 - jt0;
            } else {
                const int off = (t - n_win) * BN + 1;
                c_lo = 0; u_lo = 0; n_lo = 0;
                c_hi = nvis - off; n_hi = nvis0 - off; u_hi = nvis31 - off;
            }
            PLM(1);
            bool act[2], full[2];
            uint32_t vm[2];                                    // per-thread validity bits of a partial chunk
            if (n_lo <= 0 && n_hi >= BN - 1) {                 // most tiles: every row of the warp sees every column
                act[0] = act[1] = full[0] = full[1] = true;
                vm[0] = vm[1] = 0xffffffffu;
            } else {
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
            }
            if (STREAM && t >= n_win) {
                // the tile's 64 leave times, two per lane, are passed round the warp and tested against this row's position
                // (shared memory has no room for a scratch at two CTAs per SM); the chunks take the masked path
                const int e0 = (t - n_win) * BN;
                const int32_t* lvp = leave + (size_t)bhk * R;
                const int l0 = e0 + lane < R ? lvp[e0 + lane] : 0, l1 = e0 + 32 + lane < R ? lvp[e0 + 32 + lane] : 0;
                uint32_t m0 = 0, m1 = 0;
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    m0 |= (__shfl_sync(0xffffffffu, l0, c) > i ? 1u : 0u) << c;
                    m1 |= (__shfl_sync(0xffffffffu, l1, c) > i ? 1u : 0u) << c;
                }
                vm[0] &= m0; vm[1] &= m1;
                full[0] = full[1] = false;
            }
            PLM(2);
            mbar_wait(bar_s0 + 8 * (t & 1), (t >> 1) & 1, 3);  // S(t) is in TMEM buffer t & 1
            tc_fence_after();
            PLM(3);
            gather_issue(t + KST, false, rk);                  // its stage held K(t), which S(t) has finished reading
            PLM(4);
            const uint32_t s_col = (t & 1) * BN;
            uint32_t r[2][32];
#pragma unroll
            for (int cb = 0; cb < 2; ++cb)
                if (act[cb]) tmem_ld32(tmem + lane_base + s_col + cb * 32, r[cb]);
            tmem_wait_ld();
            PLM(5);
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
            // lazy rescale: the running max only moves when the new one is far above it (exp2 arguments stay <= 8)
            PLM(6);
            float alpha = 1.f;
            bool need = false;
            if (m_run == -INFINITY) m_run = m_tile;             // nothing accumulated yet for this row: O row is 0
            else if (m_tile > m_run + 8.f) { alpha = fast_exp2(m_run - m_tile); m_run = m_tile; need = true; }
            if (__any_sync(0xffffffffu, need)) {
                // PV(t-1) must be done before O is rescaled
                if (t > 0) { mbar_wait(((t - 1) & 1) ? bar_pv1 : bar_pv0, ((t - 1) >> 1) & 1, 4); tc_fence_after(); }
#pragma unroll 1
                for (int cb = 0; cb < D / 32 + (S::ONES ? 1 : 0); ++cb) {   // (rolled: rarely taken, and the softmax loop is sensitive to its code size)   // with ONES the row-sum columns are rescaled too
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
            PLM(7);
            const float neg_m = m_run == -INFINITY ? 0.f : -m_run;
            uint64_t ls2[2] = {0ull, 0ull};                    // two chains of packed pairs
            const uint64_t c2p = pack2(c2, c2), nmp = pack2(neg_m, neg_m);
            uint32_t pk[32];                                   // the row of P as 64 bf16, two per word
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                if (act[cb]) {
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        // masked entries hold -inf: fma gives -inf and exp2(-inf) = 0.  Scale and shift of two columns
                        // are one packed fma, their contribution to the row sum one packed add
                        float a0, a1;
                        unpack2(fma2(pack2(__uint_as_float(r[cb][c]), __uint_as_float(r[cb][c + 1])), c2p, nmp), a0, a1);
                        const float p0 = fast_exp2(a0), p1 = fast_exp2(a1);
                        if (!S::ONES) ls2[(c >> 1) & 1] = add2(ls2[(c >> 1) & 1], pack2(p0, p1));   // with ONES the tensor core sums the rounded probabilities
                        __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                        pk[cb * 16 + (c >> 1)] = *reinterpret_cast<uint32_t*>(&h);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 16; ++c) pk[cb * 16 + c] = 0u;
                }
            }
            {
                float s0, s1, s2, s3;
                unpack2(ls2[0], s0, s1); unpack2(ls2[1], s2, s3);
                l_run += (s0 + s1) + (s2 + s3);
            }
            // P goes back into TMEM, over the first 32 columns of the S buffer it was computed from (this thread has
            // all of its row in registers), and feeds the PV product as the A operand: no trip through shared memory
            PLM(8);
            tmem_st32(tmem + lane_base + s_col, pk);
            tmem_wait_st();
            tc_fence_before();                                 // our TMEM accesses are ordered before the arrive
            PLM(9);
            // (P and PV barriers come in pairs by tile parity: the MMA warp consumes P(t) before it issues S(t+2), which the
            // softmax needs before it can post P(t+2) on the same barrier, so no barrier runs two phases ahead of a waiter)
            if (!compact && t > 0) mbar_wait(((t - 1) & 1) ? bar_pv1 : bar_pv0, ((t - 1) >> 1) & 1, 4);   // (the value gather below needs PV(t-1) done)
            mbar_arrive((t & 1) ? bar_p1 : bar_p0);
            PLM(10);
            // value tile t+VST-1 goes into the stage of V(t-1), which PV(t-1) has finished reading
            if (t > 0) gather_issue(t + VST - 1, true, rv);
            PLM(11);
        }
        mbar_wait(((n_tiles - 1) & 1) ? bar_pv1 : bar_pv0, ((n_tiles - 1) >> 1) & 1, 5);
        PLM_TILE(0);
        PLM(12);
        tc_fence_after();

        // ---- epilogue: O / l -> bf16, logsumexp ----------------------------------------------------------
        if (S::ONES) {                                         // the row sum is column D of the accumulator
            uint32_t q4[32];
            tmem_ld32(tmem + lane_base + O_COL + D, q4);
            tmem_wait_ld();
            l_run = __uint_as_float(q4[0]);
        }
        const float inv = 1.f / l_run;
        // the normalised rows go into the Q tile's buffer (idle: every product of the CTA has completed) in the swizzled
        // layout and leave as one tile store per warp and 64 columns (rows past the end are clipped by the tensor map;
        // a 256-byte store per thread kept the load/store unit busy for thousands of cycles)
#pragma unroll
        for (int cb = 0; cb < D / 32; ++cb) {
            uint32_t q4[32];
            tmem_ld32(tmem + lane_base + O_COL + cb * 32, q4);
            tmem_wait_ld();
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                uint32_t w4[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(q4[g * 8 + 2 * u]) * inv,
                                                             __uint_as_float(q4[g * 8 + 2 * u + 1]) * inv);
                    w4[u] = *reinterpret_cast<uint32_t*>(&h);
                }
                const int ch = (cb & 1) * 4 + g;               // 16-byte chunk within the 64-column sub-tile cb >> 1
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sQ + (cb >> 1) * 16384 + tid * 128 + ((ch ^ (tid & 7)) << 4)),
                             "r"(w4[0]), "r"(w4[1]), "r"(w4[2]), "r"(w4[3]) : "memory");
            }
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0 && i0 + warp * 32 < Tlen) {
#pragma unroll
            for (int sb = 0; sb < SUB; ++sb) tma_store_3d(&tmO, sQ + sb * 16384 + warp * 4096, sb * 64, i0 - qoff + warp * 32, bh);
            bulk_commit();
            bulk_wait_read0();                                 // the buffer is released with the CTA
        }
        if (i < Tlen) lse[(size_t)bh * (Tlen - qoff) + (i - qoff)] = m_run * 0.6931471805599453f + logf(l_run);
        PLM(13);
        PLM_FLUSH(0, 14);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, TMEM_COLS);
}

// Retained rows into contiguous tensors kc, vc [B*H][R][d] (list order; rows past the head's count are zero), so that the
// attention kernels can fetch retained tiles as TMA boxes instead of gathering rows (Section 3.1.3: the retained keys
// and values are compacted into a contiguous span when the cache is filled).  Block (32-row part, head).
__global__ void prefill_compact_kernel(const uint4* __restrict__ k, const uint4* __restrict__ v, const int32_t* __restrict__ idx,
                                       const int32_t* __restrict__ cnt, uint4* __restrict__ kc, uint4* __restrict__ vc, int Tlen,
                                       int R, int pieces)
{
    pdl_launch_dependents();
    pdl_wait();
    const int bhk = blockIdx.y, n = cnt[bhk];
    const int e_lo = blockIdx.x * 32, e_hi = min(e_lo + 32, R);
    for (int x = e_lo * pieces + threadIdx.x; x < e_hi * pieces; x += blockDim.x) {
        const int e = x / pieces, c = x - e * pieces;
        uint4 a = make_uint4(0, 0, 0, 0), b = a;
        if (e < n) {
            const size_t src = ((size_t)bhk * Tlen + idx[(size_t)bhk * R + e]) * pieces + c;
            a = k[src]; b = v[src];
        }
        kc[((size_t)bhk * R + e) * pieces + c] = a;
        vc[((size_t)bhk * R + e) * pieces + c] = b;
    }
}

template <int D>
int run(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx, const int32_t* cnt, void* o,
        float* lse, void* ws, size_t ws_bytes, cudaStream_t st, const int32_t* leave)
{
    CUtensorMap tq, tk, tv, to, tkc, tvc;
    const int BHK = p.B * p.H, BH = BHK * p.G;                 // key/value heads, query heads
    const int Tq = p.T - p.qoff;                               // query rows
    if (!make_map(&tq, q, BH, Tq, D, BM) || !make_map(&tk, k, BHK, p.T, D, BN) || !make_map(&tv, v, BHK, p.T, D, BN) ||
        !make_map(&to, o, BH, Tq, D, 32))
        return LTE_ERR_CUDA;
    // with a workspace the retained rows are compacted first and every tile is a TMA box
    const size_t half = prefill_compact_bytes(p) / 2;
    const int compact = (ws != nullptr && half > 0 && ws_bytes >= 2 * half && ((uintptr_t)ws & 127u) == 0) ? 1 : 0;
    tkc = tk; tvc = tv;
    if (compact) {
        char* kc = (char*)ws; char* vc = kc + half;
        if (int e = launch_prefill_compact(p, k, v, idx, cnt, kc, vc, st)) return e;
        if (!make_map(&tkc, kc, BHK, p.R, D, BN) || !make_map(&tvc, vc, BHK, p.R, D, BN)) return LTE_ERR_CUDA;
    }
    static PerDeviceOnce attr;
    if (int e = attr.run([] {
            cudaError_t a = cudaFuncSetAttribute(prefill_long_kernel<D, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::BYTES);
            if (a == cudaSuccess) a = cudaFuncSetAttribute(prefill_long_kernel<D, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::BYTES);
            return a != cudaSuccess ? a : cudaFuncSetAttribute(prefill_long_kernel<D, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::BYTES);
        })) return e;
    dim3 grid((Tq + BM - 1) / BM, BH);
    if (leave != nullptr) {
        if (!compact) return LTE_ERR_UNSUPPORTED;             // the streaming variant takes compacted rows only
        return cuda_status(launch_pdl(prefill_long_kernel<D, true, true>, grid, dim3(NTHREADS), Smem<D>::BYTES, st, tq, tk, tv, to, tkc, tvc,
                                      (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, idx, cnt, leave, (__nv_bfloat16*)o, lse, p.T, p.W, p.R,
                                      p.scale, p.G, p.qoff));
    }
    if (compact)
        return cuda_status(launch_pdl(prefill_long_kernel<D, true, false>, grid, dim3(NTHREADS), Smem<D>::BYTES, st, tq, tk, tv, to, tkc, tvc,
                                      (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, idx, cnt, leave, (__nv_bfloat16*)o, lse, p.T, p.W, p.R,
                                      p.scale, p.G, p.qoff));
    return cuda_status(launch_pdl(prefill_long_kernel<D, false, false>, grid, dim3(NTHREADS), Smem<D>::BYTES, st, tq, tk, tv, to, tkc, tvc,
                                  (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, idx, cnt, leave, (__nv_bfloat16*)o, lse, p.T, p.W, p.R,
                                  p.scale, p.G, p.qoff));
}

}  // namespace

// bytes of the two compacted tensors (keys, then values), each a multiple of 128; 0 where there is nothing to compact
size_t prefill_compact_bytes(const Params& p)
{
    if (p.dtype != LTE_BF16 || (p.d != 32 && p.d != 64 && p.d != 128) || p.R <= 0) return 0;
    const size_t one = ((size_t)p.B * p.H * p.R * p.d * 2 + 127) / 128 * 128;
    return 2 * one;
}

int launch_prefill_compact(const Params& p, const void* k, const void* v, const int32_t* idx, const int32_t* cnt, void* kc, void* vc,
                           cudaStream_t st)
{
    dim3 grid((p.R + 31) / 32, p.B * p.H);
    return cuda_status(launch_pdl(prefill_compact_kernel, grid, dim3(256), 0, st, (const uint4*)k, (const uint4*)v, idx, cnt, (uint4*)kc,
                                  (uint4*)vc, p.T, p.R, p.d * 2 / 16));
}

int launch_prefill_tc_long(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx,
                           const int32_t* cnt, void* o, float* lse, void* ws, size_t ws_bytes, cudaStream_t st, const int32_t* leave)
{
    if (p.d != 128) return LTE_ERR_UNSUPPORTED;
    return run<128>(p, q, k, v, idx, cnt, o, lse, ws, ws_bytes, st, leave);
}

#ifdef LTE_PROFILE
extern "C" void lte_plprof_read(unsigned long long* out, int clear)
{
    cudaMemcpyFromSymbol(out, g_plprof, sizeof(unsigned long long) * 64);
    if (clear) { unsigned long long z[64] = {}; cudaMemcpyToSymbol(g_plprof, z, sizeof(z)); }
}
#endif

int prefill_long_status_fetch_and_clear() { return status_fetch_and_clear(g_prefill_long_status); }

}  // namespace lte
