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
//                  the scale folded in), P written as bf16 into swizzled shared memory
//   O += P V       tcgen05.mma with V as an MN-major operand, accumulated in TMEM; the accumulator is rescaled
//                  in place only when a row's maximum grows by more than 2^8 (lazy rescale)
// Loads run two to three tiles ahead of the tensor core.  Every mbarrier wait is bounded; a wait that runs out
// records a status word and the kernel still terminates.
#include "tma_util.cuh"

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
constexpr uint32_t kSpinLimit = 1u << 22;

// ---- PTX wrappers -----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls, records `code`, and lets the kernel run on to its end.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, int code) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return;
        // once any wait has given up, the launch is lost: stop waiting everywhere so it ends quickly
        if ((i & 1023u) == 1023u && *reinterpret_cast<volatile int*>(&g_prefill_status) != 0) return;
    }
    atomicExch(&g_prefill_status, code);
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int x, int y, int z, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
                 "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                   "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                   "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
                 : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row atoms of 1024 bytes.
//   K-major operand  (rows = M or N index, 128 bytes of K per row): SBO = 1024 between 8-row groups.
//   MN-major operand (rows = K index, 128 bytes = 64 elements of N per row): SBO = 1024 between 8-row
//   K groups, LBO = distance between consecutive 64-element N groups.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, A K-major, B K-major or MN-major, M x N.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

template <int D> struct Smem {
    static constexpr int SUB = D / 64;                        // 64-column (128-byte) sub-tiles per row
    static constexpr int KST = D == 64 ? 3 : 2;               // key stages
    static constexpr int VST = D == 64 ? 3 : 2;               // value stages
    static constexpr int QTILE = BM * D * 2;                  // [128][D] bf16
    static constexpr int KVTILE = BN * D * 2;                 // [64][D] bf16
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = QTILE;
    static constexpr int OFF_V = OFF_K + KST * KVTILE;
    static constexpr int OFF_P = OFF_V + VST * KVTILE;        // [128][64] bf16 = 16 KB
    static constexpr int OFF_BAR = OFF_P + BM * BN * 2;       // mbarriers, tmem slot
    static constexpr int OFF_IDX = OFF_BAR + 128;             // 128 staged list entries
    static constexpr int BYTES = OFF_IDX + 512;
    static constexpr uint32_t TMEM_COLS = 256;                // S0: [0,64)  S1: [64,128)  O: [128, 128+D)
};

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void softmax_group_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ uint64_t desc64(uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | lo; }

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
    const uint32_t sQ = base + S::OFF_Q, sK = base + S::OFF_K, sV = base + S::OFF_V, sP = base + S::OFF_P;
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
            constexpr uint32_t IDESC_O = instr_desc(BM, D, true);
            // descriptor words: lo = (address >> 4) | LBO field, hi = SBO field | version | swizzle mode
            constexpr uint32_t HI = (1024u >> 4) | (1u << 14) | (2u << 29);
            const uint32_t q_lo = (sQ >> 4) | (1u << 16), k_lo = (sK >> 4) | (1u << 16), p_lo = (sP >> 4) | (1u << 16);
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
                    const uint32_t vb = v_lo + (uint32_t)(t % VST) * (S::KVTILE >> 4);
#pragma unroll
                    for (int kk = 0; kk < BN / 16; ++kk)
                        umma(tmem + O_COL, desc64(p_lo + kk * 2, HI), desc64(vb + kk * 128, HI), IDESC_O, (t > 0 || kk > 0) ? 1u : 0u);
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

        const float c2 = scale * 1.4426950408889634f;          // logits are handled in the log2 domain: x = s * c2
        const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;   // this warp's TMEM lanes
        float m_run = -INFINITY, l_run = 0.f;                  // running max (log2 domain) and sum

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
                    for (int c = 0; c < 32; ++c) mr[c & 3] = fmaxf(mr[c & 3], __uint_as_float(r[cb][c]));
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
                for (int cb = 0; cb < D / 32; ++cb) {
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
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                uint32_t pk[16];
                if (act[cb]) {
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        // masked entries hold -inf: fma gives -inf and exp2(-inf) = 0
                        const float p0 = fast_exp2(fmaf(__uint_as_float(r[cb][c]), c2, neg_m));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(r[cb][c + 1]), c2, neg_m));
                        ls[(c >> 1) & 3] += p0 + p1;
                        __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                        pk[c >> 1] = *reinterpret_cast<uint32_t*>(&h);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 16; ++c) pk[c] = 0u;
                }
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int ch = cb * 4 + g;
                    const uint32_t dst = sP + tid * 128 + ((ch ^ (tid & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[4 * g]), "r"(pk[4 * g + 1]),
                                 "r"(pk[4 * g + 2]), "r"(pk[4 * g + 3]) : "memory");
                }
            }
            l_run += (ls[0] + ls[1]) + (ls[2] + ls[3]);
            fence_proxy_async();                               // P (generic proxy) -> visible to the MMA (async proxy)
            tc_fence_before();                                 // our TMEM reads of S(t) are ordered before the arrive
            mbar_arrive(bar_p);
            PROF(9 + 6 * t);
        }
        PROF(50);
        mbar_wait(bar_pv, (n_tiles - 1) & 1, 5);
        tc_fence_after();
        PROF(51);

        // ---- epilogue: O / l -> bf16, logsumexp ----------------------------------------------------------
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
