// Prefill attention on the 5th-generation tensor cores (Section 3.1.3, "Cached prefilling and decoding").
//
// One CTA (128 threads) per 128-query tile of one (b,h).  Key/value tiles of 128 rows come from two
// sources, as in the paper's two-stage loop: (1) the contiguous window span, staged by TMA
// (cp.async.bulk.tensor, 128-byte swizzle); (2) the retained rows already out of the tile's window,
// gathered row by row with cp.async into the same swizzled layout (idx is ascending, so the entries a
// query may see are a prefix of the list and every mask is a column range).  Per tile:
//   S = Q K^T      tcgen05.mma (kind::f16, bf16 in, fp32 out) into TMEM, operands from shared memory
//   softmax        thread r owns query row r = TMEM lane r: tcgen05.ld, range mask, running max / sum in
//                  fp32 (exp2 with the scale folded in), P written as bf16 into swizzled shared memory
//   O_tile = P V   tcgen05.mma with V as an MN-major operand, fresh TMEM accumulator, then folded into
//                  the fp32 register accumulator with the online-softmax rescale.
// K/V loads of tile t+1 are in flight while tile t is computed (two stages).  Every mbarrier wait is
// bounded; a wait that runs out records a status word and the kernel still terminates.
#include "tma_util.cuh"

namespace lte {

__device__ int g_prefill_status = 0;          // 0 = fine; otherwise the code of the wait that gave up

#ifdef LTE_PROFILE
__device__ long long g_prof[64];
#define PROF(slot) do { if (blockIdx.x == 5 && blockIdx.y == 3 && threadIdx.x == 64) g_prof[slot] = clock64(); } while (0)
#else
#define PROF(slot) do { } while (0)
#endif

namespace {

constexpr int BM = 128, BN = 64, NTHREADS = 128;
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
    static constexpr int QTILE = BM * D * 2;                  // [128][D] bf16
    static constexpr int KVTILE = BN * D * 2;                 // [64][D] bf16
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = QTILE;                       // 2 stages
    static constexpr int OFF_V = OFF_K + 2 * KVTILE;          // 2 stages
    static constexpr int OFF_P = OFF_V + 2 * KVTILE;          // [128][64] bf16 = 16 KB
    static constexpr int OFF_BAR = OFF_P + BM * BN * 2;       // mbarriers, tmem slot, scratch ints
    static constexpr int OFF_IDX = OFF_BAR + 128;             // 128 staged list entries
    static constexpr int BYTES = OFF_IDX + 512;
    static constexpr uint32_t TMEM_COLS = D == 64 ? 128 : 256; // S: [0,64), O: [64, 64+D)
};

template <int D>
__global__ void __launch_bounds__(NTHREADS, D == 64 ? 3 : 2)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const __nv_bfloat16* __restrict__ kg,
                  const __nv_bfloat16* __restrict__ vg, const int32_t* __restrict__ idx,
                  const int32_t* __restrict__ cnt, __nv_bfloat16* __restrict__ o, float* __restrict__ lse, int Tlen,
                  int W, int R, float scale)
{
    using S = Smem<D>;
    constexpr int SUB = S::SUB;
    constexpr uint32_t TMEM_COLS = S::TMEM_COLS;
    constexpr uint32_t O_COL = BN;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 1023u) != 0) {                                 // the swizzled tiles need 1024-byte alignment
        if (threadIdx.x == 0) atomicExch(&g_prefill_status, 9);
        return;
    }
    PROF(0);
    const uint32_t sQ = base + S::OFF_Q, sK = base + S::OFF_K, sV = base + S::OFF_V, sP = base + S::OFF_P;
    const uint32_t bar_q = base + S::OFF_BAR, bar_k0 = bar_q + 8, bar_v0 = bar_q + 24, bar_s = bar_q + 40;
    const uint32_t tmem_slot = bar_q + 48;
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_raw + S::OFF_BAR + 48);
    volatile int* s_nvmax = reinterpret_cast<volatile int*>(smem_raw + S::OFF_BAR + 52);
    volatile int* s_idx = reinterpret_cast<volatile int*>(smem_raw + S::OFF_IDX);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.y;
    const int i0 = blockIdx.x * BM;
    const int i = i0 + tid;                                    // this thread's query row
    const int i_hi = min(i0 + BM - 1, Tlen - 1);

    if (tid == 0) {
        mbar_init(bar_q, 1); mbar_init(bar_k0, 1); mbar_init(bar_k0 + 8, 1); mbar_init(bar_v0, 1);
        mbar_init(bar_v0 + 8, 1); mbar_init(bar_s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) { __syncwarp(); tmem_alloc(tmem_slot, TMEM_COLS); }
    __syncthreads();
    if (tid == 0) {
        mbar_expect_tx(bar_q, S::QTILE);
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb) tma_load_3d(sQ + sb * 16384, &tmQ, sb * 64, i0, bh, bar_q);
    }

    PROF(1);
    // ---- retained entries visible to this row: idx ascending => a prefix of length nvis.  The list is
    // staged through shared memory 128 entries at a time and searched there.
    const int32_t* id = idx + (size_t)bh * R;
    const int n_ret = cnt[bh];
    const int lim = min(i, Tlen - 1) - W;                      // entry visible iff idx <= lim
    const int lim_max = i_hi - W;
    int nvis = 0;
    for (int e0 = 0; e0 < n_ret; e0 += 128) {
        const int n_here = min(128, n_ret - e0);
        __syncthreads();
        if (tid < n_here) s_idx[tid] = id[e0 + tid];
        __syncthreads();
        if (s_idx[n_here - 1] <= lim) nvis += n_here;
        else {
            int lo = 0, hi = n_here;
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (s_idx[mid] <= lim) lo = mid + 1; else hi = mid; }
            nvis += lo;
        }
        if (s_idx[n_here - 1] > lim_max) break;                // uniform: nothing further is visible to any row
    }
    if (i == i_hi) *s_nvmax = nvis;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;
    const int nv_max = *s_nvmax;
    PROF(2);

    const int j_start = max(i0 - W + 1, 0);
    const int n_win = (i_hi - j_start + 1 + BN - 1) / BN;
    const int n_rt = (nv_max + BN - 1) / BN;
    const int n_tiles = n_win + n_rt;

    // ---- loads: K and V of a tile are tracked separately (K runs two tiles ahead, V one) -----------------
    auto issue_kv = [&](int t, bool is_v) {
        if (t >= n_tiles) return;
        const int st = t & 1;
        const uint32_t dst = (is_v ? sV : sK) + st * S::KVTILE;
        if (t < n_win) {
            if (tid == 0) {
                const uint32_t bar = (is_v ? bar_v0 : bar_k0) + 8 * st;
                mbar_expect_tx(bar, S::KVTILE);
                const int y = j_start + t * BN;
#pragma unroll
                for (int sb = 0; sb < SUB; ++sb) tma_load_3d(dst + sb * 8192, is_v ? &tmV : &tmK, sb * 64, y, bh, bar);
            }
        } else {
            // gather: two threads per row, each copies half of the row's 16-byte chunks
            const int row = tid & 63, part = tid >> 6;
            const int e = (t - n_win) * BN + row;
            const bool ok = e < nv_max;
            const __nv_bfloat16* src = (is_v ? vg : kg) + ((size_t)bh * Tlen + (ok ? id[e] : 0)) * D;
            const uint32_t nbytes = ok ? 16u : 0u;             // rows past the visible prefix are zero-filled
#pragma unroll
            for (int c = 0; c < D / 16; ++c) {
                const int ch = part * (D / 16) + c;
                const uint32_t off = (ch >> 3) * 8192 + row * 128 + (((ch & 7) ^ (row & 7)) << 4);
                cp_async16(dst + off, src + ch * 8, nbytes);
            }
        }
    };

    issue_kv(0, false); issue_kv(1, false); issue_kv(0, true);
    cp_async_commit();

    constexpr uint32_t IDESC_S = instr_desc(BM, BN, false);
    constexpr uint32_t IDESC_O = instr_desc(BM, D, true);
    const float c2 = scale * 1.4426950408889634f;              // logits are handled in the log2 domain: x = s * c2
    const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;   // this warp's TMEM lanes
    uint32_t k_phase = 0, v_phase = 0;                         // bit st = parity of that stage's TMA barrier

    auto mma_s = [&](int t) {                                  // thread 0 only
        const int st = t & 1;
        if (t < n_win) { mbar_wait(bar_k0 + 8 * st, (k_phase >> st) & 1u, 2); k_phase ^= 1u << st; }
        const uint32_t kb = sK + st * S::KVTILE;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk)
            umma(tmem, smem_desc(sQ + (kk >> 2) * 16384 + (kk & 3) * 32, 16, 1024),
                 smem_desc(kb + (kk >> 2) * 8192 + (kk & 3) * 32, 16, 1024), IDESC_S, kk > 0);
        umma_commit(bar_s);
    };

    // first S: needs Q and K(0)
    cp_async_wait<0>();
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
        tc_fence_after();
        mbar_wait(bar_q, 0, 1);
        mma_s(0);
    }

    PROF(3);
    float m_run = -INFINITY, l_run = 0.f;                      // running max (log2 domain) and sum

    for (int t = 0; t < n_tiles; ++t) {
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
        uint32_t vm[2];                                        // per-thread validity bits of a partial chunk
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
            const int lo = cb * 32, hi = lo + 31;
            act[cb] = lo <= u_hi && hi >= u_lo;
            full[cb] = lo >= n_lo && hi <= n_hi;
            const int a = min(max(c_lo - lo, 0), 32), b = min(max(c_hi - lo + 1, 0), 32);
            const uint32_t below_b = b >= 32 ? 0xffffffffu : ((1u << b) - 1u);
            const uint32_t below_a = a >= 32 ? 0xffffffffu : ((1u << a) - 1u);
            vm[cb] = b > a ? (below_b & ~below_a) : 0u;
        }

        PROF(4 + 6 * t);
        mbar_wait(bar_s, t & 1, 3);                            // S(t) is in TMEM; PV(t-1) has completed too
        tc_fence_after();
        PROF(5 + 6 * t);
        issue_kv(t + 2, false); issue_kv(t + 1, true);
        cp_async_commit();
        PROF(6 + 6 * t);

        uint32_t r[2][32];
#pragma unroll
        for (int cb = 0; cb < 2; ++cb)
            if (act[cb]) tmem_ld32(tmem + lane_base + cb * 32, r[cb]);
        tmem_wait_ld();
        PROF(7 + 6 * t);
        float m_raw = -INFINITY;                               // row max of the raw logits (scale applied after)
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
            if (!act[cb]) continue;
            if (full[cb]) {
#pragma unroll
                for (int c = 0; c < 32; ++c) m_raw = fmaxf(m_raw, __uint_as_float(r[cb][c]));
            } else {
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const float x = (vm[cb] & (1u << c)) ? __uint_as_float(r[cb][c]) : -INFINITY;
                    r[cb][c] = __float_as_uint(x);
                    m_raw = fmaxf(m_raw, x);
                }
            }
        }
        const float m_tile = m_raw * c2;
        // lazy rescale: the running max only moves when the new one is far above it (exp2 arguments stay <= 8)
        float alpha = 1.f;
        bool need = false;
        if (m_run == -INFINITY) m_run = m_tile;                 // nothing accumulated yet for this row: O row is 0
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
        float l_tile = 0.f;
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
            uint32_t pk[16];
            if (act[cb]) {
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    // masked entries hold -inf: fma gives -inf and exp2(-inf) = 0
                    const float p0 = fast_exp2(fmaf(__uint_as_float(r[cb][c]), c2, neg_m));
                    const float p1 = fast_exp2(fmaf(__uint_as_float(r[cb][c + 1]), c2, neg_m));
                    l_tile += p0 + p1;
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
        l_run += l_tile;
        PROF(8 + 6 * t);

        cp_async_wait<1>();                                    // gathered K(t+1), V(t) have landed
        fence_proxy_async();                                   // P and gathered rows -> visible to the MMA proxy
        tc_fence_before();
        __syncthreads();
        PROF(9 + 6 * t);
        if (tid == 0) {
            tc_fence_after();
            const int st = t & 1;
            if (t < n_win) { mbar_wait(bar_v0 + 8 * st, (v_phase >> st) & 1u, 4); v_phase ^= 1u << st; }
            const uint32_t vb = sV + st * S::KVTILE;
#pragma unroll
            for (int kk = 0; kk < BN / 16; ++kk)
                umma(tmem + O_COL, smem_desc(sP + kk * 32, 16, 1024), smem_desc(vb + kk * 2048, 8192, 1024), IDESC_O,
                     (t > 0 || kk > 0) ? 1u : 0u);
            if (t + 1 < n_tiles) mma_s(t + 1);
            else umma_commit(bar_s);                           // final: signals that the last PV is done
        }
    }
    PROF(50);
    mbar_wait(bar_s, n_tiles & 1, 5);
    tc_fence_after();
    PROF(51);

    // ---- epilogue: O / l -> bf16, logsumexp --------------------------------------------------------------
    {
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
    }
    PROF(52);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
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
extern "C" int lte_prof_read(long long* out) { return cudaMemcpyFromSymbol(out, g_prof, sizeof(long long) * 64) == cudaSuccess ? 0 : -1; }
#endif

int prefill_status_fetch_and_clear()
{
    int h = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&h, g_prefill_status, sizeof(int)) != cudaSuccess) return -1;
    if (h != 0) cudaMemcpyToSymbol(g_prefill_status, &zero, sizeof(int));
    return h;
}

}  // namespace lte
