// Prefill attention on the 5th-generation tensor cores (Section 3.1.3, "Cached prefilling and decoding").
//
// Persistent CTAs (two per SM): each walks work items, an item being one 128-query tile of one (b,h), so that the
// loads of the next item are in flight while the current one is finished (a CTA per item spent a third of its life
// waiting for its first tiles).  Four softmax warps, one MMA-issue warp and one load warp.  Key/value tiles of 64
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
// Tiles are numbered through all items of a CTA (g); stage, buffer and barrier phase of a tile follow from g alone.
// Every mbarrier wait is bounded; a wait that runs out records a status word and the kernel still terminates.
#include "tc_common.cuh"

namespace lte {

__device__ StatusWord g_prefill_status = LTE_STATUS_INIT;         // 0 = fine; otherwise the code of the wait that gave up

// -DLTE_PROFILE: cycle counters of the row threads' phases (lane 0 of warp 0 of every CTA), added up over all CTAs;
// PP(c) charges the time since the previous mark to phase c.  The product build does not define it.
#ifdef LTE_PROFILE
__device__ unsigned long long g_pprof[16];
__device__ unsigned long long g_pprof_cta[1024 * 2];           // per CTA: globaltimer at kernel entry and at the end of the row loop
#define PP_DECL long long pp_t = clock64(); long long pp_a[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}
#define PP(c) do { const long long pp_n = clock64(); pp_a[c] += pp_n - pp_t; pp_t = pp_n; } while (0)
#define PP_COUNT(c, n) do { pp_a[c] += (n); } while (0)
#define PP_FLUSH() do { if (warp == 0 && lane == 0) { _Pragma("unroll") for (int pp_i = 0; pp_i < 16; ++pp_i) atomicAdd(&g_pprof[pp_i], (unsigned long long)pp_a[pp_i]); \
    unsigned long long gt; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt)); if (blockIdx.x < 1024) g_pprof_cta[blockIdx.x * 2 + 1] = gt; } } while (0)
#else
#define PP_DECL
#define PP(c)
#define PP_COUNT(c, n)
#define PP_FLUSH()
#endif

namespace {

constexpr int BM = 128, BN = 64, NTHREADS = 192;
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
    // d = 64: the row sums are taken by the tensor core as well: PV gets 16 extra B columns of ones, so column D of
    // the accumulator is sum_j P_ij of exactly the (bf16-rounded) probabilities the product used.  The ones live in one
    // more 64-column group, LBO away from the value tile.
    static constexpr bool ONES = D == 64;
    static constexpr int OFF_ONES = OFF_V + VST * KVTILE;     // [64][64] bf16 ones (8 KB), d = 64 only
    static constexpr int OFF_BAR = OFF_ONES + (ONES ? BN * 128 : 0);   // mbarriers, tmem slot
    static constexpr int OFF_LV = OFF_BAR + 256;              // STREAM: the leave times of a retained tile, [4 warps][64]
    static constexpr int BYTES = OFF_LV + 4 * 64 * 4;
    static constexpr uint32_t TMEM_COLS = 256;                // S0: [0,64)  S1: [64,128)  O: [128, 128+D) (+16 row-sum columns)
};

// One work item: a 128-query tile of one (b,h).
struct Item {
    int bh, bhk, i0, i_hi, j_start, n_win;              // bh: query head (b, h, g); bhk: its key/value head (b, h)
};
// Items are numbered from the last query tile of every (b,h) down to the first: later query tiles see more retained
// rows and cost more, and a CTA takes items n, n + grid, n + 2 grid, ... so every CTA gets one item of each cost band
// (largest first), which balances the static schedule.
__device__ __forceinline__ Item decode_item(int item, int n_qt, int n_bh, int Tlen, int W, int G, int qoff)
{
    Item it;
    const int r = item / n_bh;
    it.bh = item - r * n_bh;
    it.bhk = it.bh / G;                                 // the G query heads of a key/value head are adjacent
    it.i0 = qoff + (n_qt - 1 - r) * BM;                 // positions; the query tensors start at position qoff
    it.i_hi = min(it.i0 + BM - 1, Tlen - 1);
    it.j_start = max(it.i0 - W + 1, 0);
    it.n_win = (it.i_hi - it.j_start + 1 + BN - 1) / BN;
    return it;
}
// Entries of the ascending list id[0, n) that are <= lim (whole warp).
__device__ __forceinline__ int count_le(const int32_t* id, int n, int lim, int lane)
{
    int c = 0;
    for (int e0 = 0; e0 < n; e0 += 32) {
        const int e = e0 + lane < n ? id[e0 + lane] : 0x7fffffff;
        const unsigned bal = __ballot_sync(0xffffffffu, e <= lim);
        c += __popc(bal);
        if (bal != 0xffffffffu) break;
    }
    return c;
}

// Warps 0-3 (128 threads): softmax (thread r owns query row r) and the cp.async gathers of retained rows.
// Warp 4, one lane: every tcgen05.mma.  Warp 5, one lane: the TMA loads of Q and of the window tiles (a single
// lane doing both was the bottleneck: its dependent instruction stream took longer per tile than the softmax).
// They meet on mbarriers (g = the tile's number within the CTA, it = the item's):
//   bar_q                    Q of item `it` has landed (TMA)                          phase it
//   bar_qf    (commit)       the last S product of item `it` has completed            phase it     MMA -> load
//   bar_of    (4 arrivals)   O of item `it` has been read out of TMEM                 phase it     softmax -> MMA
//   bar_s[b]  (commit)       S(g) is in TMEM buffer b = g & 1                         phase g >> 1 MMA -> softmax
//   bar_p     (4 arrivals)   P(g) is in TMEM, over S(g)                               phase g      softmax -> MMA
//   bar_pv    (commit)       PV(g) has completed                                      phase g      MMA -> softmax
//   bar_g[b]  (4 arrivals)   gathers issued before the top of tile g have landed      phase g >> 1 softmax -> MMA
//   bar_k[s], bar_v[s]       TMA transaction barriers of the window tiles (one phase per TMA use of the stage)
//   bar_kf[s], bar_vf[s]     (commit) the MMA that read the stage's tile g has completed   phase g / stages   MMA -> load
// S(g+1) and S(g+2) are computed while the softmax of tile g runs; loads run two to three tiles ahead, across items.
// COMPACT: the retained rows were copied into contiguous tensors [B*H][R][d] beforehand (tmKc, tmVc), so retained tiles are
// TMA boxes like the window tiles and the softmax warps gather nothing (a compile-time variant: the gather code costs the
// softmax loop instruction-cache room even where it does not run).
// STREAM (with COMPACT): the list is every entry that is retained at some query of a chunk, and entry e is gone from query
// leave[e] on (the streaming reading of a chunk): retained tiles take one more mask, leave > query position.
template <int D, bool COMPACT, bool STREAM>
__global__ void __launch_bounds__(NTHREADS, 2)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV,
                  const __grid_constant__ CUtensorMap tmKc, const __grid_constant__ CUtensorMap tmVc,
                  const __nv_bfloat16* __restrict__ kg,
                  const __nv_bfloat16* __restrict__ vg, __nv_bfloat16* __restrict__ og, const int32_t* __restrict__ idx,
                  const int32_t* __restrict__ cnt, const int32_t* __restrict__ leave, float* __restrict__ lse, int Tlen,
                  int W, int R, float scale, int n_qt, int n_bh, int G, int qoff, int dg)
{
    const int n_items = n_qt * n_bh;
#ifdef LTE_PROFILE
    if (threadIdx.x == 0 && blockIdx.x < 1024) { unsigned long long gt; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt)); g_pprof_cta[blockIdx.x * 2] = gt; }
#endif
    using S = Smem<D>;
    constexpr int SUB = S::SUB, KST = S::KST, VST = S::VST;
    constexpr uint32_t TMEM_COLS = S::TMEM_COLS;
    constexpr uint32_t O_COL = 2 * BN;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 1023u) != 0) {                                 // the swizzled tiles need 1024-byte alignment
        if (threadIdx.x == 0) atomicExch(&g_prefill_status.code, 9);
        return;
    }
    const uint32_t sQ = base + S::OFF_Q, sK = base + S::OFF_K, sV = base + S::OFF_V;
    const uint32_t bar_q = base + S::OFF_BAR;
    const uint32_t bar_k0 = bar_q + 8;                         // 3 slots
    const uint32_t bar_v0 = bar_q + 32;                        // 3 slots
    const uint32_t bar_s0 = bar_q + 56;                        // 2 slots
    const uint32_t bar_g0 = bar_q + 72;                        // 2 slots
    const uint32_t bar_p = bar_q + 88, bar_pv = bar_q + 96;
    const uint32_t bar_kf0 = bar_q + 104;                      // 3 slots: K stage free
    const uint32_t bar_vf0 = bar_q + 128;                      // 3 slots: V stage free
    const uint32_t bar_qf = bar_q + 152, bar_of = bar_q + 160;
    const uint32_t tmem_slot = bar_q + 168;
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_raw + S::OFF_BAR + 168);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        mbar_init(bar_q, 1);
#pragma unroll
        for (int s2 = 0; s2 < 3; ++s2) {
            mbar_init(bar_k0 + 8 * s2, 1); mbar_init(bar_v0 + 8 * s2, 1);
            mbar_init(bar_kf0 + 8 * s2, 1); mbar_init(bar_vf0 + 8 * s2, 1);
        }
        mbar_init(bar_s0, 1); mbar_init(bar_s0 + 8, 1);
        // the softmax warps arrive once per warp (lane 0, after __syncwarp): 128 arrivals on one barrier word serialise
        mbar_init(bar_g0, 4); mbar_init(bar_g0 + 8, 4);
        mbar_init(bar_p, 4); mbar_init(bar_pv, 1);
        mbar_init(bar_qf, 1); mbar_init(bar_of, 4);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) tmem_alloc(tmem_slot, TMEM_COLS);
    if (S::ONES && tid < 128) {                                // 8 KB of bf16 1.0: 64 bytes per thread, once per CTA
#pragma unroll
        for (int u = 0; u < 4; ++u)
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base + S::OFF_ONES + tid * 64 + u * 16), "r"(0x3F803F80u) : "memory");
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;
    pdl_launch_dependents();
    pdl_wait();                                                // everything above ran beside the previous kernel's tail

    if (warp == 5) {
        // ================================= load warp (lane 0 issues) ========================================
        uint32_t g = 0;                                        // tiles of the items before this one
        int it = 0;
        for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++it) {
            const Item w = decode_item(item, n_qt, n_bh, Tlen, W, G, qoff);
            if (lane == 0) {
                // Q: its buffer is free once the previous item's last S product has completed
                if (it > 0) mbar_wait(bar_qf, (it - 1) & 1, 12);
                mbar_expect_tx(bar_q, S::QTILE);
#pragma unroll
                for (int sb = 0; sb < SUB; ++sb) tma_load_3d(sQ + sb * 16384, &tmQ, sb * 64, w.i0 - qoff, w.bh, bar_q);
            }
            // tiles, each into its stage as soon as the MMA that read the stage's previous tile has completed
            auto load_tiles = [&](int t_lo, int t_hi) {
                for (int t = t_lo; t < t_hi; ++t) {
                    const uint32_t gg = g + t;
                    const bool win = t < w.n_win;
                    const int y = win ? w.j_start + t * BN : (t - w.n_win) * BN;
                    const uint32_t ks = gg % KST, vs = gg % VST;
                    if (gg >= (uint32_t)KST) mbar_wait(bar_kf0 + 8 * ks, (gg / KST - 1) & 1u, 6);
                    mbar_expect_tx(bar_k0 + 8 * ks, S::KVTILE);
#pragma unroll
                    for (int sb = 0; sb < SUB; ++sb)
                        tma_load_3d(sK + ks * S::KVTILE + sb * 8192, win ? &tmK : &tmKc, sb * 64, y, w.bhk, bar_k0 + 8 * ks);
                    if (gg >= (uint32_t)VST) mbar_wait(bar_vf0 + 8 * vs, (gg / VST - 1) & 1u, 8);
                    mbar_expect_tx(bar_v0 + 8 * vs, S::KVTILE);
#pragma unroll
                    for (int sb = 0; sb < SUB; ++sb)
                        tma_load_3d(sV + vs * S::KVTILE + sb * 8192, win ? &tmV : &tmVc, sb * 64, y, w.bhk, bar_v0 + 8 * vs);
                }
            };
            if (lane == 0) load_tiles(0, w.n_win);
            // the item's retained tiles also take tile numbers (counted after the window loads are on their way)
            const int n_ret_tiles = (count_le(idx + (size_t)w.bhk * R, cnt[w.bhk], w.i_hi - W, lane) + BN - 1) / BN;
            if (COMPACT && lane == 0) load_tiles(w.n_win, w.n_win + n_ret_tiles);
            g += w.n_win + n_ret_tiles;
        }
    } else if (warp == 4) {
        // ================================= MMA warp (lane 0 issues) =========================================
        // The whole warp walks the loop and waits on the barriers; only the tcgen05 instructions are guarded by the lane
        // test.  Descriptors and addresses are then computed in convergent code (the compiler can keep them in uniform
        // registers), which roughly halves the issue cost of an MMA compared with a loop run by one lane alone.
        constexpr uint32_t IDESC_S = instr_desc(BM, BN, false);
        constexpr uint32_t IDESC_O = S::ONES ? instr_desc(BM, D + 16, true) : instr_desc(BM, D, true);
        // descriptor words: lo = (address >> 4) | LBO field, hi = SBO field | version | swizzle mode
        constexpr uint32_t HI = (1024u >> 4) | (1u << 14) | (2u << 29);
        const uint32_t q_lo = (sQ >> 4) | (1u << 16), k_lo = (sK >> 4) | (1u << 16);
        uint32_t g = 0, g_waited = 0;                          // tiles before this item; bar_g phases consumed
        uint32_t k_par = 0, v_par = 0;                         // TMA barrier parities (bit per stage)
        int it = 0;
        // tiles of an item (whole warp: the count of visible list entries takes global loads)
        auto item_tiles = [&](int item) {
            if (item >= n_items) return 0;
            const Item w = decode_item(item, n_qt, n_bh, Tlen, W, G, qoff);
            return w.n_win + (count_le(idx + (size_t)w.bhk * R, cnt[w.bhk], w.i_hi - W, lane) + BN - 1) / BN;
        };
        int n_tiles_next = item_tiles(blockIdx.x);
        for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++it) {
            const Item w = decode_item(item, n_qt, n_bh, Tlen, W, G, qoff);
            const int n_tiles = n_tiles_next;
            int ts = 0;                                        // S products of this item issued so far
            // gathers issued before the top of tile gg have landed
            auto need_g = [&](uint32_t gg) {
                while (g_waited <= gg) { mbar_wait(bar_g0 + 8 * (g_waited & 1), (g_waited >> 1) & 1, 10); ++g_waited; }
            };
            auto mma_s = [&]() {                           // S of the item's tile ts
                const uint32_t gg = g + ts, ks = gg % KST;
                if (COMPACT || ts < w.n_win) { mbar_wait(bar_k0 + 8 * ks, (k_par >> ks) & 1u, 2); k_par ^= 1u << ks; }
                else need_g(g + max(ts - (KST == 2 ? 1 : 2), 0));   // a gathered K tile: issued in tile ts - KST or in the item's prologue
                tc_fence_after();
                const uint32_t kb = k_lo + ks * (S::KVTILE >> 4);
                const uint32_t dcol = tmem + (gg & 1) * BN;
                ++ts;
                if (lane == 0) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        umma(dcol, desc64(q_lo + (kk >> 2) * 1024 + (kk & 3) * 2, HI), desc64(kb + (kk >> 2) * 512 + (kk & 3) * 2, HI),
                             IDESC_S, kk > 0);
                    umma_commit(bar_s0 + 8 * (gg & 1));
                    umma_commit(bar_kf0 + 8 * ks);             // the K stage is free once this S has completed
                    if (ts == n_tiles) umma_commit(bar_qf);    // and so is Q after the item's last S
                }
                __syncwarp();
            };

            mbar_wait(bar_q, it & 1, 1);
            mma_s();                                           // tile 0 is always a window tile
            if (n_tiles > 1) mma_s();
            // the next item's tile count, fetched while the softmax of this item's first tile runs
            n_tiles_next = item_tiles(item + gridDim.x);
            {
                for (int t = 0; t < n_tiles; ++t) {
                    const uint32_t gg = g + t, vs = gg % VST;
                    if (!COMPACT) need_g(gg);
                    if (COMPACT || t < w.n_win) { mbar_wait(bar_v0 + 8 * vs, (v_par >> vs) & 1u, 4); v_par ^= 1u << vs; }
                    // value operand: the second 64-column group of B is the next sub-tile (d = 128) or the block of
                    // ones (d = 64, LBO = its distance from the value stage)
                    const uint32_t va = sV + vs * S::KVTILE;
                    const uint32_t vb = (va >> 4) | ((S::ONES ? ((base + S::OFF_ONES - va) >> 4) : (8192u >> 4)) << 16);
                    if (t == 0 && it > 0) mbar_wait(bar_of, (it - 1) & 1, 13);   // the previous item's O has been read out
                    mbar_wait(bar_p, gg & 1, 7);
                    tc_fence_after();
                    if (lane == 0) {
#pragma unroll
                        for (int kk = 0; kk < BN / 16; ++kk)
                            umma_ts(tmem + O_COL, tmem + (gg & 1) * BN + kk * 8, desc64(vb + kk * 128, HI), IDESC_O, (t > 0 || kk > 0) ? 1u : 0u);
                        umma_commit(bar_pv);
                        umma_commit(bar_vf0 + 8 * vs);         // the V stage is free once PV has completed
                    }
                    __syncwarp();
                    // S two tiles ahead, into the S buffer the softmax has just released
                    if (ts < n_tiles) mma_s();
                }
            }
            g += n_tiles;
            __syncwarp();
        }
    } else {
        // =================================== softmax warps ==================================================
        const float c2 = scale * 1.4426950408889634f;          // logits are handled in the log2 domain: x = s * c2
        const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;   // this warp's TMEM lanes
        const int g_row = tid >> 3, g_sub = tid & 7;           // gathers: 8 lanes per row, 16 rows per pass
        uint32_t g = 0;                                        // tiles of the items before this one
        int it = 0;
        // the list length and the first 128 list entries of an item are fetched one item ahead, so that the visible
        // counts at the start of an item wait for no load (entries past cnt are never used: the length guards them)
        int pf_cnt = 0, pf_e[4] = {0, 0, 0, 0};
        auto prefetch_list = [&](int item) {
            if (item < n_items) {
                const Item w = decode_item(item, n_qt, n_bh, Tlen, W, G, qoff);
                pf_cnt = cnt[w.bhk];
#pragma unroll
                for (int u = 0; u < 4; ++u) pf_e[u] = u * 32 + lane < R ? idx[(size_t)w.bhk * R + u * 32 + lane] : 0x7fffffff;
            }
        };
        prefetch_list(blockIdx.x);
        PP_DECL;
        for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++it) {
            const Item w = decode_item(item, n_qt, n_bh, Tlen, W, G, qoff);
            const int bh = w.bh, bhk = w.bhk, n_win = w.n_win, j_start = w.j_start;
            const int32_t* id = idx + (size_t)bhk * R;
            const int n_ret = pf_cnt;
            const int i = w.i0 + tid;                          // this thread's query row
            // retained entries visible to this row.  The rows of a warp are consecutive and the list is ascending, so
            // nvis(row) = #{idx <= lim of lane 0} + #{idx in (lim of lane 0, lim of this lane]}: a ballot count plus a
            // 31-bit map of the entries that fall between the warp's first and last limit.  No block barrier.
            const int lim = min(i, Tlen - 1) - W;              // entry visible iff idx <= lim
            const int lim_max = w.i_hi - W;
            const int lim0 = __shfl_sync(0xffffffffu, lim, 0), lim31 = __shfl_sync(0xffffffffu, lim, 31);
            int nvis = 0, nv_max = 0;                          // nv_max: entries visible to the tile's last row
            {
                uint32_t bits = 0;
                for (int e0 = 0; e0 < n_ret; e0 += 128) {
                    int e[4];
                    if (e0 == 0) {
#pragma unroll
                        for (int u = 0; u < 4; ++u) e[u] = u * 32 + lane < n_ret ? pf_e[u] : 0x7fffffff;
                    } else {
#pragma unroll
                        for (int u = 0; u < 4; ++u) e[u] = e0 + u * 32 + lane < n_ret ? id[e0 + u * 32 + lane] : 0x7fffffff;
                    }
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
            const int nvis_first = __shfl_sync(0xffffffffu, nvis, 0), nvis_last = __shfl_sync(0xffffffffu, nvis, 31);
            prefetch_list(item + gridDim.x);
            PP(0); PP_COUNT(14, 1); PP_COUNT(15, n_tiles);

            // gather of one retained tile (t = its number within the item): 8 lanes per row copy its 16-byte chunks
            // (coalesced reads, conflict-free swizzled writes); rows past the visible prefix are zero-filled
            auto gather_rows = [&](int t, int (&rows4)[4]) {   // row positions of this thread's 4 rows of tile t
#pragma unroll
                for (int ps = 0; ps < 4; ++ps) {
                    const int e = (t - n_win) * BN + ps * 16 + g_row;
                    rows4[ps] = (t >= n_win && t < n_tiles && e < nv_max) ? id[e] : -1;
                }
            };
            auto gather_issue = [&](int t, bool is_v, const int (&rows4)[4]) {
                if (t >= n_win && t < n_tiles) {
                    const uint32_t st = is_v ? ((g + t) % VST) : ((g + t) % KST);
                    const uint32_t dst = (is_v ? sV : sK) + st * S::KVTILE;
#pragma unroll
                    for (int ps = 0; ps < 4; ++ps) {
                        const int row = ps * 16 + g_row;
                        const bool ok = rows4[ps] >= 0;
                        const __nv_bfloat16* src = (is_v ? vg : kg) + ((size_t)bhk * Tlen + (ok ? rows4[ps] : 0)) * dg;
#pragma unroll
                        for (int c = g_sub; c < D / 8; c += 8) {
                            const uint32_t off = (c >> 3) * 8192 + row * 128 + (((c & 7) ^ (row & 7)) << 4);
                            const bool real = ok && c * 8 < dg;    // columns past the head dimension are zero-filled
                            cp_async16(dst + off, src + (real ? c * 8 : 0), real ? 16u : 0u);
                        }
                    }
                }
                cp_async_commit();
            };
            // prologue gathers: the first KST key tiles and VST value tiles, where those are retained tiles.  Their
            // stages are free: every product of the previous item has completed (its last bar_s and bar_pv were awaited).
            if (!COMPACT && n_win < KST) {
                int rows4[4];
                for (int t = 0; t < KST; ++t) { gather_rows(t, rows4); gather_issue(t, false, rows4); }
                for (int t = 0; t < VST; ++t) { gather_rows(t, rows4); gather_issue(t, true, rows4); }
            }
            float m_run = -INFINITY, l_run = 0.f;              // running max (log2 domain) and sum (sum only if !ONES)
            bool gathered = !COMPACT && n_win < KST;           // some gather of this item may be in flight (warp-uniform)

            for (int t = 0; t < n_tiles; ++t) {
                const uint32_t gg = g + t;
                // row positions for this tile's two gathers, fetched first so their latency hides under the softmax
                // (all of this tile's gather work sits behind warp-uniform tests: most tiles of a short list have none)
                const bool k_gather = !COMPACT && t + KST >= n_win && t + KST < n_tiles;
                const bool v_gather = !COMPACT && t > 0 && t + VST - 1 >= n_win && t + VST - 1 < n_tiles;
                int rk[4], rv[4];
                if (k_gather) gather_rows(t + KST, rk);
                if (v_gather) gather_rows(t + VST - 1, rv);
                if (!COMPACT) {
                    // gathers issued before this point have landed (all of them, or all but the latest value tile)
                    if (gathered) {
                        if (VST == 3) cp_async_wait<1>(); else cp_async_wait<0>();
                        fence_proxy_async();
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_g0 + 8 * (gg & 1));
                }

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
                // rows of a warp are consecutive and both bounds grow with the row: the bounds of its first and last row
                // give the warp's union range (columns any row sees) and intersection range (columns every row sees).
                // They follow from the warp's first row alone (no shuffles on the per-tile path).
                int u_lo, u_hi, n_lo, n_hi;
                if (t < n_win) {
                    const int jt0 = j_start + t * BN, ia = i - lane, ib = ia + 31;
                    u_lo = max(ia - W + 1, 0) - jt0; n_lo = max(ib - W + 1, 0) - jt0;
                    n_hi = ia - jt0; u_hi = ib - jt0;
                } else {
                    u_lo = n_lo = 0;
                    n_hi = nvis_first - (t - n_win) * BN - 1; u_hi = nvis_last - (t - n_win) * BN - 1;
                }
                bool act[2], full[2];
                uint32_t vm[2];                                // per-thread validity bits of a partial chunk
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
                if (STREAM && t >= n_win) {
                    // the tile's 64 leave times go through a per-warp scratch (two coalesced loads), then every row tests
                    // them against its own position; the chunks take the masked path
                    int* slv = reinterpret_cast<int*>(smem_raw + S::OFF_LV) + warp * 64;
                    const int e0 = (t - n_win) * BN;
                    const int32_t* lvp = leave + (size_t)bhk * R;
                    __syncwarp();                              // the previous tile's readers are done
                    slv[lane] = e0 + lane < R ? lvp[e0 + lane] : 0;
                    slv[32 + lane] = e0 + 32 + lane < R ? lvp[e0 + 32 + lane] : 0;
                    __syncwarp();
#pragma unroll
                    for (int cb = 0; cb < 2; ++cb) {
                        uint32_t m = 0;
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            const int4 l4 = *reinterpret_cast<const int4*>(&slv[cb * 32 + c]);
                            m |= (l4.x > i ? 1u : 0u) << c; m |= (l4.y > i ? 2u : 0u) << c;
                            m |= (l4.z > i ? 4u : 0u) << c; m |= (l4.w > i ? 8u : 0u) << c;
                        }
                        vm[cb] &= m;
                        full[cb] = false;
                    }
                }
                PP(1);
                mbar_wait(bar_s0 + 8 * (gg & 1), (gg >> 1) & 1, 3);   // S is in TMEM buffer gg & 1
                tc_fence_after();
                PP(2);
                if (k_gather) { gather_issue(t + KST, false, rk); gathered = true; }   // its stage held this tile's K, which S has finished reading
                else if (!COMPACT) cp_async_commit();
                const uint32_t s_col = (gg & 1) * BN;
                uint32_t r[2][32];
#pragma unroll
                for (int cb = 0; cb < 2; ++cb)
                    if (act[cb]) tmem_ld32(tmem + lane_base + s_col + cb * 32, r[cb]);
                tmem_wait_ld();
                PP(3);
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
                float alpha = 1.f;
                bool need = false;
                if (m_run == -INFINITY) m_run = m_tile;         // nothing accumulated yet for this row: O row is 0
                else if (m_tile > m_run + 8.f) { alpha = fast_exp2(m_run - m_tile); m_run = m_tile; need = true; }
                if (__any_sync(0xffffffffu, need)) {
                    // PV of the previous tile must be done before O is rescaled
                    if (t > 0) { mbar_wait(bar_pv, (gg - 1) & 1, 4); tc_fence_after(); }
#pragma unroll 1
                    for (int cb = 0; cb < D / 32 + (S::ONES ? 1 : 0); ++cb) {   // with ONES the row-sum columns are rescaled too (rolled: rarely taken, and the loop is sensitive to its code size)
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
                PP(4);
                const uint64_t c2_2 = pack2(c2, c2), neg_m2 = pack2(neg_m, neg_m);
                float ls[4] = {0.f, 0.f, 0.f, 0.f};
                uint32_t pk[32];                               // the row of P as 64 bf16, two per word
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
                    if (act[cb]) {
#pragma unroll
                        for (int c = 0; c < 32; c += 2) {
                            // masked entries hold -inf: fma gives -inf and exp2(-inf) = 0
                            float x0, x1;                      // two columns per packed fp32 instruction
                            unpack2(fma2(pack2(__uint_as_float(r[cb][c]), __uint_as_float(r[cb][c + 1])), c2_2, neg_m2), x0, x1);
                            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
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
                PP(5);
                // P goes back into TMEM, over the first 32 columns of the S buffer it was computed from (this thread has
                // all of its row in registers), and feeds the PV product as the A operand: no trip through shared memory
                tmem_st32(tmem + lane_base + s_col, pk);
                tmem_wait_st();
                tc_fence_before();                             // our TMEM accesses are ordered before the arrive
                // PV of the previous tile has normally completed long ago.  Every phase of bar_pv is awaited in turn (a
                // parity test is only meaningful for the current or the previous phase), and before the arrive: after
                // it the barrier could run ahead of this thread.  At t = 0 the item's epilogue has awaited it.
                PP(6);
                if (t > 0) mbar_wait(bar_pv, (gg - 1) & 1, 4);
                PP(7);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_p);
                // value tile t+VST-1 goes into the stage of tile t-1's V, which that PV has finished reading
                if (v_gather) { gather_issue(t + VST - 1, true, rv); gathered = true; }
                else if (!COMPACT) cp_async_commit();
            }
            PP(1);
            mbar_wait(bar_pv, (g + n_tiles - 1) & 1, 5);
            tc_fence_after();
            PP(8);

            // ---- epilogue: O / l -> bf16, logsumexp ------------------------------------------------------
            if (S::ONES) {                                     // the row sum is column D of the accumulator
                uint32_t q1;
                tmem_ld1(tmem + lane_base + O_COL + D, q1);
                tmem_wait_ld();
                l_run = __uint_as_float(q1);
            }
            const float inv = 1.f / l_run;
            // a normalised row is D * 2 contiguous bytes of the output (whole 128-byte lines, and the rows of a warp are
            // consecutive): each thread stores its own row with 16-byte stores, no staging in shared memory
            __nv_bfloat16* orow = og + ((size_t)bh * (Tlen - qoff) + (i - qoff)) * dg;
#pragma unroll
            for (int sb = 0; sb < SUB; ++sb) {
                uint32_t ow[32];                               // 64 columns of the row as bf16 pairs
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
                    uint32_t q4[32];
                    tmem_ld32(tmem + lane_base + O_COL + sb * 64 + cb * 32, q4);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(q4[c]) * inv, __uint_as_float(q4[c + 1]) * inv);
                        ow[cb * 16 + (c >> 1)] = *reinterpret_cast<uint32_t*>(&h);
                    }
                }
                if (sb == SUB - 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_of);        // the accumulator may take the next item
                }
                PP(9);
                if (i < Tlen) {
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch)
                        if (sb * 64 + ch * 8 < dg)
                            *reinterpret_cast<uint4*>(orow + sb * 64 + ch * 8) = make_uint4(ow[4 * ch], ow[4 * ch + 1], ow[4 * ch + 2], ow[4 * ch + 3]);
                }
            }
            if (i < Tlen) lse[(size_t)bh * (Tlen - qoff) + (i - qoff)] = m_run * 0.6931471805599453f + logf(l_run);
            g += n_tiles;
            PP(11);
        }
        PP_FLUSH();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, TMEM_COLS);
}

template <int D>
int run(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx, const int32_t* cnt, void* o,
        float* lse, void* ws, size_t ws_bytes, cudaStream_t st, const int32_t* leave)
{
    CUtensorMap tq, tk, tv, tkc, tvc;
    const int BHK = p.B * p.H, BH = BHK * p.G;                 // key/value heads, query heads
    const int Tq = p.T - p.qoff;                               // query rows (the whole sequence unless a chunk is prefilled)
    // head dimension in memory: D, or half of it (d = 32 runs the d = 64 kernel: the tensor maps' 64-column boxes reach past
    // the 32 columns a row has and the copy engine fills the rest of every tile row with zeros, which change no product)
    const int dg = p.d;
    if (!make_map(&tq, q, BH, Tq, dg, BM) || !make_map(&tk, k, BHK, p.T, dg, BN) || !make_map(&tv, v, BHK, p.T, dg, BN)) return LTE_ERR_CUDA;
    // with a workspace the retained rows are compacted first and every tile is a TMA box
    const size_t half = prefill_compact_bytes(p) / 2;
    const bool compact = ws != nullptr && half > 0 && ws_bytes >= 2 * half && ((uintptr_t)ws & 127u) == 0;
    tkc = tk; tvc = tv;
    if (compact) {
        char* kc = (char*)ws; char* vc = kc + half;
        if (int e = launch_prefill_compact(p, k, v, idx, cnt, kc, vc, st)) return e;
        if (!make_map(&tkc, kc, BHK, p.R, dg, BN) || !make_map(&tvc, vc, BHK, p.R, dg, BN)) return LTE_ERR_CUDA;
    }
    static PerDeviceOnce attr;
    if (int e = attr.run([] {
            cudaError_t a = cudaFuncSetAttribute(prefill_tc_kernel<D, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::BYTES);
            if (a == cudaSuccess) a = cudaFuncSetAttribute(prefill_tc_kernel<D, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::BYTES);
            return a != cudaSuccess ? a : cudaFuncSetAttribute(prefill_tc_kernel<D, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::BYTES);
        })) return e;
    int sms = 0;
    if (int e = device_sm_count(&sms)) return e;
    const int slots = 2 * sms;                                 // resident CTAs: two per SM
    const int n_qt = (Tq + BM - 1) / BM, n_items = n_qt * BH;
    const int grid = n_items < slots ? n_items : slots;
    if (leave != nullptr) {
        if (!compact) return LTE_ERR_UNSUPPORTED;             // the streaming variant takes compacted rows only
        return cuda_status(launch_pdl(prefill_tc_kernel<D, true, true>, dim3(grid), dim3(NTHREADS), Smem<D>::BYTES, st, tq, tk, tv, tkc, tvc,
                                      (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (__nv_bfloat16*)o, idx, cnt, leave, lse, p.T, p.W, p.R,
                                      p.scale, n_qt, BH, p.G, p.qoff, dg));
    }
    if (compact)
        return cuda_status(launch_pdl(prefill_tc_kernel<D, true, false>, dim3(grid), dim3(NTHREADS), Smem<D>::BYTES, st, tq, tk, tv, tkc, tvc,
                                      (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (__nv_bfloat16*)o, idx, cnt, leave, lse, p.T, p.W, p.R,
                                      p.scale, n_qt, BH, p.G, p.qoff, dg));
    return cuda_status(launch_pdl(prefill_tc_kernel<D, false, false>, dim3(grid), dim3(NTHREADS), Smem<D>::BYTES, st, tq, tk, tv, tkc, tvc,
                                  (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (__nv_bfloat16*)o, idx, cnt, leave, lse, p.T, p.W, p.R,
                                  p.scale, n_qt, BH, p.G, p.qoff, dg));
}

}  // namespace

// leave: null, or the streaming reading's per-entry leave times (d = 64 or 128 with a workspace: the tiled kernels; otherwise
// the row-by-row kernel)
int launch_prefill_tc(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx,
                      const int32_t* cnt, void* o, float* lse, void* ws, size_t ws_bytes, cudaStream_t st, const int32_t* leave)
{
    if (p.d == 64 || p.d == 32) {
        const int e = run<64>(p, q, k, v, idx, cnt, o, lse, ws, ws_bytes, st, leave);
        if (e != LTE_ERR_UNSUPPORTED || leave == nullptr) return e;
    }
    if (leave != nullptr) {
        if (p.d == 128) {
            const int e = launch_prefill_tc_long(p, q, k, v, idx, cnt, o, lse, ws, ws_bytes, st, leave);
            if (e != LTE_ERR_UNSUPPORTED) return e;
        }
        return launch_prefill_simt(p, q, k, v, idx, cnt, o, lse, st, leave);
    }
    // d = 128: ten and more key tiles per item; one CTA per item under the hardware scheduler is faster there
    if (p.d == 128) return launch_prefill_tc_long(p, q, k, v, idx, cnt, o, lse, ws, ws_bytes, st);
    return launch_prefill_simt(p, q, k, v, idx, cnt, o, lse, st);
}


#ifdef LTE_PROFILE
extern "C" int lte_pprof_read(unsigned long long* out, int clear)
{
    if (cudaMemcpyFromSymbol(out, g_pprof, sizeof(unsigned long long) * 16) != cudaSuccess) return -1;
    if (clear) { unsigned long long z[16] = {}; cudaMemcpyToSymbol(g_pprof, z, sizeof(z)); }
    return 0;
}
extern "C" int lte_pprof_cta_read(unsigned long long* out)
{
    return cudaMemcpyFromSymbol(out, g_pprof_cta, sizeof(unsigned long long) * 2048) == cudaSuccess ? 0 : -1;
}
#endif

int prefill_status_fetch_and_clear()
{
    const int h = status_fetch_and_clear(g_prefill_status), h2 = prefill_long_status_fetch_and_clear();
    return h != 0 ? h : h2;
}

}  // namespace lte
