// Retention logits of the single-layer scorer (Section 3.1.1): z_j = bias + sum_t <w_t, x_{j+t-half}>.
//
// Each input row x_p = [k_p ; v_p] is read from HBM once per tile and turned into K partial dot
// products Y[p][t] = <w_t, x_p> by one thread (weights broadcast from shared memory, fp32 FMA);
// the logit of token j is then the shifted diagonal sum_t Y[j+t-half][t], taken from shared memory.
// A block of NT threads covers NT rows and emits NT-(K-1) logits; the K-1 halo rows are recomputed by
// the neighbouring block.  HBM traffic: 2*d elements read and one fp32 written per token and head.
#include "tc_common.cuh"

namespace lte {

__device__ StatusWord g_scores_status = LTE_STATUS_INIT;

namespace {

constexpr int NT = 128;

template <typename T> struct Vec16;   // 16-byte vector of T as floats
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static void load(const __nv_bfloat16* p, float (&f)[8]) {
        uint4 u = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};
template <> struct Vec16<float> {
    static constexpr int N = 4;
    __device__ static void load(const float* p, float (&f)[4]) {
        float4 u = __ldg(reinterpret_cast<const float4*>(p));
        f[0] = u.x; f[1] = u.y; f[2] = u.z; f[3] = u.w;
    }
};

template <typename T, int D, int K>
__global__ void __launch_bounds__(NT) scores_kernel(const T* __restrict__ k, const T* __restrict__ v,
                                                    const float* __restrict__ w, const float* __restrict__ bias,
                                                    float* __restrict__ z, float* __restrict__ r, int H, int Tlen)
{
    constexpr int HALF = K / 2;
    constexpr int TJ = NT - (K - 1);
    constexpr int VN = Vec16<T>::N;
    __shared__ __align__(16) float ws[K * 2 * D];
    __shared__ float ys[NT * K];

    const int bh = blockIdx.y;
    const int h = bh % H;
    const int j0 = blockIdx.x * TJ;
    const int tid = threadIdx.x;
    for (int i = tid; i < K * 2 * D; i += NT) ws[i] = w[(size_t)h * K * 2 * D + i];
    __syncthreads();

    const int p = j0 - HALF + tid;          // input row of this thread
    float acc[K];
#pragma unroll
    for (int t = 0; t < K; ++t) acc[t] = 0.f;
    if (p >= 0 && p < Tlen) {
        const T* rows[2] = {k + ((size_t)bh * Tlen + p) * D, v + ((size_t)bh * Tlen + p) * D};
#pragma unroll
        for (int part = 0; part < 2; ++part) {
#pragma unroll 2
            for (int c = 0; c < D; c += VN) {
                float x[VN];
                Vec16<T>::load(rows[part] + c, x);
#pragma unroll
                for (int t = 0; t < K; ++t) {
                    const float4* wv = reinterpret_cast<const float4*>(&ws[(t * 2 + part) * D + c]);
#pragma unroll
                    for (int u = 0; u < VN / 4; ++u) {
                        float4 ww = wv[u];
                        acc[t] = fmaf(x[4 * u + 0], ww.x, acc[t]);
                        acc[t] = fmaf(x[4 * u + 1], ww.y, acc[t]);
                        acc[t] = fmaf(x[4 * u + 2], ww.z, acc[t]);
                        acc[t] = fmaf(x[4 * u + 3], ww.w, acc[t]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int t = 0; t < K; ++t) ys[tid * K + t] = acc[t];
    __syncthreads();

    const int j = j0 + tid;
    if (tid < TJ && j < Tlen) {
        float zz;
        if (j + HALF > Tlen - 1) {
            zz = -INFINITY;                 // right context does not exist yet
        } else {
            zz = bias ? bias[h] : 0.f;
#pragma unroll
            for (int t = 0; t < K; ++t) zz += ys[(tid + t) * K + t];
        }
        z[(size_t)bh * Tlen + j] = zz;
        if (r) r[(size_t)bh * Tlen + j] = 1.f / (1.f + __expf(-zz));
    }
}

// ---- bf16, d = 64 or 128: TMA-staged tiles, the K partial dot products per row on the tensor cores -----------------
// Y[p][t] = <w_t, x_p> for a tile of 128 input rows is the small GEMM  X[128 x 2d] * Wt[2d x K]:
//   A = the tile of k rows, then of v rows, exactly as TMA delivers them (128-byte swizzle, K-major); rows left of
//       position 0 or right of T-1 arrive as zeros, which is the scorer's zero padding;
//   B = the fp32 weights split into three bf16 pieces (hi + mid + lo reproduces all 24 mantissa bits, and
//       bf16 x bf16 products are exact in the fp32 accumulator), one B row per (piece, tap), built in shared memory;
//   D = fp32 in TMEM; the thread owning row p adds the three pieces and the block takes the shifted diagonal sum.
// HBM is touched by the copy engine only; the kernel is bound by HBM bandwidth, not by the fp32 ALUs.
using namespace tc;
#ifdef LTE_PROFILE
__device__ long long g_sprof[64];
#define SPROF(slot) do { if (blockIdx.x == 5 && threadIdx.x == 64 && (slot) < 64) g_sprof[slot] = clock64(); } while (0)
#else
#define SPROF(slot) do { } while (0)
#endif

template <int D, int K> struct ScoresTc {
    static constexpr int SUB = D / 64;
    static constexpr int NB = (3 * K + 15) / 16 * 16;    // B rows = accumulator columns (multiple of 16)
    static constexpr int NSTAGE = D == 64 ? 3 : 2;       // input-tile stages (each: k tile + v tile)
    static constexpr int STAGE = 2 * SUB * 16384;
    static constexpr int B_SLOT = NB * 128;              // bytes of one [NB][64] sub-tile of B (a multiple of 1024)
    static constexpr int OFF_B = NSTAGE * STAGE, OFF_YS = OFF_B + 2 * SUB * B_SLOT, OFF_BAR = OFF_YS + NT * K * 4;
    static constexpr int BYTES = OFF_BAR + 96;
    static constexpr uint32_t ACC_COLS = NB <= 32 ? 32 : 64;   // columns of one accumulator buffer (two buffers)
};

// A CTA walks `tiles_per_cta` consecutive row tiles of one (b,h): B is built once, the input tiles stream through an
// NSTAGE ring (TMA), the MMA of tile i+1 runs while the threads take tile i out of TMEM (two accumulator buffers).
template <int D, int K>
__global__ void __launch_bounds__(NT + 64) scores_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                       const __grid_constant__ CUtensorMap tmV,
                                                       const float* __restrict__ w, const float* __restrict__ bias,
                                                       float* __restrict__ z, float* __restrict__ r, int H, int Tlen,
                                                       int n_flat, int dg)
{
    // dg = the head dimension in memory: D, or D / 2 = 32 for the d = 64 kernel on d = 32 data (the tensor maps then fill
    // the upper half of every tile row with zeros, and B carries zeros in the same columns)
    using C = ScoresTc<D, K>;
    constexpr int HALF = K / 2;
    constexpr int TJ = NT - (K - 1);
    constexpr int SUB = C::SUB, NB = C::NB, NSTAGE = C::NSTAGE;
    constexpr uint32_t TMEM_COLS = 2 * C::ACC_COLS;
    extern __shared__ __align__(1024) uint8_t smem[];
    float* ys = reinterpret_cast<float*>(smem + C::OFF_YS);
    const uint32_t tile0 = smem_u32(smem);
    const uint32_t bar_ld0 = tile0 + C::OFF_BAR, bar_mma0 = bar_ld0 + 8 * NSTAGE, tmem_slot = bar_mma0 + 16;
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem + C::OFF_BAR + 8 * NSTAGE + 16);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int n_all = (Tlen + TJ - 1) / TJ;              // row tiles per head
    // this CTA's share of the flat list of (head, row tile) pairs: an even split, heads may change along the way
    const int f_begin = (int)(((long long)blockIdx.x * n_flat) / gridDim.x);
    const int f_end = (int)(((long long)(blockIdx.x + 1) * n_flat) / gridDim.x);
    const int n_tiles = f_end - f_begin;
    if (n_tiles <= 0) return;

    if ((tile0 & 1023u) != 0) { if (tid == 0) atomicExch(&g_scores_status.code, 8); return; }
    const uint32_t bar_free0 = tmem_slot + 8;            // 2 barriers: accumulator buffer taken out of TMEM (128 arrivals)
    const uint32_t bar_b = bar_free0 + 16;               // B rebuilt for the next head (128 arrivals)
    if (tid == 0) {
#pragma unroll
        for (int s2 = 0; s2 < NSTAGE; ++s2) mbar_init(bar_ld0 + 8 * s2, 1);
        mbar_init(bar_mma0, 1); mbar_init(bar_mma0 + 8, 1);
        mbar_init(bar_free0, 128); mbar_init(bar_free0 + 8, 128); mbar_init(bar_b, 128);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;
    pdl_launch_dependents();
    pdl_wait();                                          // everything above ran beside the previous kernel's tail

    if (warp == 5) {
        // ---- load lane: streams the input tiles through the stage ring ----------------------------------------------
        if ((tid & 31) == 0) {
            int fb = f_begin / n_all, ft = f_begin - fb * n_all;      // (head, row tile) of the next tile to load
            for (int i = 0; i < n_tiles; ++i) {
                // the stage is free once the MMAs of the tile that used it have completed
                if (i >= NSTAGE) mbar_wait_s(bar_mma0 + 8 * ((i - NSTAGE) & 1), ((i - NSTAGE) >> 1) & 1, 3, &g_scores_status);
                const uint32_t dst = tile0 + (i % NSTAGE) * C::STAGE, bar = bar_ld0 + 8 * (i % NSTAGE);
                const int y = ft * TJ - HALF;
                mbar_expect_tx(bar, C::STAGE);
#pragma unroll
                for (int sb = 0; sb < SUB; ++sb) {
                    tma_load_3d(dst + sb * 16384, &tmK, sb * 64, y, fb, bar);
                    tma_load_3d(dst + (SUB + sb) * 16384, &tmV, sb * 64, y, fb, bar);
                }
                if (++ft == n_all) { ft = 0; ++fb; }
            }
        }
    } else if (warp == 4) {
        // ---- MMA warp: the whole warp walks the loop and waits; only the tcgen05 instructions are guarded by the lane test
        //      (descriptors computed in convergent code are cheaper to issue than from a loop run by one lane alone)
        {
            const bool leader = (tid & 31) == 0;
            constexpr uint32_t IDESC = instr_desc(128, NB, false);
            const uint32_t b_lo = desc_lo(tile0 + C::OFF_B, 16), a_lo0 = desc_lo(tile0, 16);
            int ft = f_begin % n_all, n_heads = 0;
            bool new_head = true;
            for (int i = 0; i < n_tiles; ++i) {
                if (new_head) { mbar_wait_s(bar_b, n_heads & 1, 5, &g_scores_status); ++n_heads; }   // B of this head is ready
                mbar_wait_s(bar_ld0 + 8 * (i % NSTAGE), (i / NSTAGE) & 1, 7, &g_scores_status);
                if (i >= 2) mbar_wait_s(bar_free0 + 8 * (i & 1), ((i - 2) >> 1) & 1, 4, &g_scores_status);   // its accumulator buffer is free
                tc_fence_after();
                const uint32_t a_lo = a_lo0 + (uint32_t)(i % NSTAGE) * (C::STAGE >> 4);
                const uint32_t dcol = tmem + (i & 1) * C::ACC_COLS;
                if (leader) {
#pragma unroll
                    for (int kk = 0; kk < 2 * D / 16; ++kk)   // 2d input channels, 16 per instruction
                        umma(dcol, desc64(a_lo + (kk >> 2) * 1024 + (kk & 3) * 2, kDescHi),
                             desc64(b_lo + (kk >> 2) * (C::B_SLOT >> 4) + (kk & 3) * 2, kDescHi), IDESC, kk > 0);
                    umma_commit(bar_mma0 + 8 * (i & 1));
                }
                __syncwarp();
                new_head = ++ft == n_all;
                if (new_head) ft = 0;
            }
        }
    } else {
        // ---- row threads: thread p owns input row p of the tile -------------------------------------------------------
        auto group_sync = [&]() { asm volatile("bar.sync 1, 128;" ::: "memory"); };
        const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;
        int cur_bh = -1;
        float bh_bias = 0.f;
        for (int i = 0; i < n_tiles; ++i) {
            const int f = f_begin + i, bh = f / n_all, ti = f - bh * n_all;
            if (bh != cur_bh) {
                // new head: this thread has taken every earlier tile out of TMEM, and it only gets here after the others
                // did too (the group barrier at the end of the previous tile), so no MMA is still reading the old B
                cur_bh = bh;
                const int h = bh % H;
                bh_bias = bias ? bias[h] : 0.f;
                // B: row n = piece * K + t, columns = the 2d input channels (k part, then v part); zero rows above 3K
                // (one 16-byte chunk = 8 channels of one row per step; all of a thread's weights are fetched before any is
                // converted: the shared-memory stores below are compiler barriers and would serialise the load latencies)
                constexpr int NCH = NB * 2 * D / 8 / NT;        // chunks per thread
                static_assert(NB * 2 * D / 8 % NT == 0, "B chunks must divide evenly over the row threads");
                float4 wf[NCH][2];
#pragma unroll
                for (int q = 0; q < NCH; ++q) {
                    const int e = tid + q * NT, n = e / (2 * D / 8), c8 = e % (2 * D / 8);
                    wf[q][0] = wf[q][1] = make_float4(0.f, 0.f, 0.f, 0.f);
                    const int part = c8 / (D / 8), cin = (c8 % (D / 8)) * 8;   // key or value half; channel within it
                    if (n < 3 * K && cin < dg) {
                        const float4* src = reinterpret_cast<const float4*>(w + ((size_t)h * K + n % K) * 2 * dg + part * dg + cin);
                        wf[q][0] = src[0]; wf[q][1] = src[1];
                    }
                }
#pragma unroll
                for (int q = 0; q < NCH; ++q) {
                    const int e = tid + q * NT, n = e / (2 * D / 8), c8 = e % (2 * D / 8);
                    const int piece = n / K;
                    uint32_t pk[4] = {0u, 0u, 0u, 0u};
                    if (n < 3 * K) {
                        const float wv8[8] = {wf[q][0].x, wf[q][0].y, wf[q][0].z, wf[q][0].w, wf[q][1].x, wf[q][1].y, wf[q][1].z, wf[q][1].w};
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            float v2[2];
#pragma unroll
                            for (int x = 0; x < 2; ++x) {
                                const float wv = wv8[2 * u + x];
                                const float hi = __bfloat162float(__float2bfloat16_rn(wv));
                                const float mid = __bfloat162float(__float2bfloat16_rn(wv - hi));
                                const float lo = __bfloat162float(__float2bfloat16_rn((wv - hi) - mid));
                                v2[x] = piece == 0 ? hi : (piece == 1 ? mid : lo);
                            }
                            __nv_bfloat162 h2 = __floats2bfloat162_rn(v2[0], v2[1]);
                            pk[u] = *reinterpret_cast<uint32_t*>(&h2);
                        }
                    }
                    const int sub = c8 / 8, ch = c8 % 8;   // 64-column sub-tile (k: 0..SUB-1, v: SUB..2SUB-1), chunk in row
                    const uint32_t dst = tile0 + C::OFF_B + sub * C::B_SLOT + n * 128 + ((ch ^ (n & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
                }
                fence_proxy_async();
                mbar_arrive(bar_b);
            }
            SPROF(4 * i);
            mbar_wait_s(bar_mma0 + 8 * (i & 1), (i >> 1) & 1, 6, &g_scores_status);
            tc_fence_after();
            SPROF(4 * i + 1);
            {
                const uint32_t col = tmem + lane_base + (i & 1) * C::ACC_COLS;
                uint32_t acc[32];
                tmem_ld32(col, acc);
                float y[K];
                if constexpr (NB <= 32) {
                    tmem_wait_ld();
#pragma unroll
                    for (int t = 0; t < K; ++t)
                        y[t] = (__uint_as_float(acc[2 * K + t]) + __uint_as_float(acc[K + t])) + __uint_as_float(acc[t]);
                } else {
                    uint32_t acc2[32];
                    tmem_ld32(col + 32, acc2);
                    tmem_wait_ld();
#pragma unroll
                    for (int t = 0; t < K; ++t) {
                        const int i0 = t, i1 = K + t, i2 = 2 * K + t;
                        const float a0 = __uint_as_float(i0 < 32 ? acc[i0] : acc2[i0 - 32]);
                        const float a1 = __uint_as_float(i1 < 32 ? acc[i1] : acc2[i1 - 32]);
                        const float a2 = __uint_as_float(i2 < 32 ? acc[i2] : acc2[i2 - 32]);
                        y[t] = (a2 + a1) + a0;
                    }
                }
                tc_fence_before();
                mbar_arrive(bar_free0 + 8 * (i & 1));     // the accumulator buffer can take tile i + 2
#pragma unroll
                for (int t = 0; t < K; ++t) ys[tid * K + t] = y[t];
            }
            SPROF(4 * i + 2);
            group_sync();                                  // ys complete
            const int j = ti * TJ + tid;
            if (tid < TJ && j < Tlen) {
                float zz;
                if (j + HALF > Tlen - 1) {
                    zz = -INFINITY;
                } else {
                    zz = bh_bias;
#pragma unroll
                    for (int t = 0; t < K; ++t) zz += ys[(tid + t) * K + t];
                }
                z[(size_t)bh * Tlen + j] = zz;
                if (r) r[(size_t)bh * Tlen + j] = 1.f / (1.f + __expf(-zz));
            }
            group_sync();                                  // ys is rewritten by the next tile
            SPROF(4 * i + 3);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, TMEM_COLS);
}

template <int D, int K>
int run_tma(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st, int dg = D)
{
    using C = ScoresTc<D, K>;
    constexpr int TJ = NT - (K - 1);
    CUtensorMap tk, tv;
    if (!make_map(&tk, k, p.B * p.H, p.T, dg, NT) || !make_map(&tv, v, p.B * p.H, p.T, dg, NT)) return LTE_ERR_CUDA;
    static PerDeviceOnce attr;
    if (int e = attr.run([] { return cudaFuncSetAttribute(scores_tc_kernel<D, K>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::BYTES); })) return e;
    int n_sm = 0;
    if (int e = device_sm_count(&n_sm)) return e;
    // one wave of CTAs (two per SM at d = 64, one at d = 128) shares the flat list of (head, row tile) pairs evenly
    const int n_all = (p.T + TJ - 1) / TJ, BH = p.B * p.H;
    const long long n_flat = (long long)n_all * BH;
    if (n_flat > 0x7fffffffLL) return LTE_ERR_UNSUPPORTED;
    const int slots = n_sm * (D == 64 ? 2 : 1);
    const int n_cta = (int)(n_flat < slots ? n_flat : slots);
    if (launch_pdl(scores_tc_kernel<D, K>, dim3(n_cta), dim3(NT + 64), C::BYTES, st, tk, tv, p.w, p.bias, z, r, p.H, p.T,
                   (int)n_flat, dg) != cudaSuccess)
        return LTE_ERR_CUDA;
    return cuda_status(cudaGetLastError());
}

template <typename T, int D, int K>
int run(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    constexpr int TJ = NT - (K - 1);
    dim3 grid((p.T + TJ - 1) / TJ, p.B * p.H);
    scores_kernel<T, D, K><<<grid, NT, 0, st>>>((const T*)k, (const T*)v, p.w, p.bias, z, r, p.H, p.T);
    return cuda_status(cudaGetLastError());
}

template <typename T, int D, int K>
int pick(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    if constexpr (sizeof(T) == 2 && (D == 64 || D == 128)) return run_tma<D, K>(p, k, v, z, r, st);
    else if constexpr (sizeof(T) == 2 && D == 32) return run_tma<64, K>(p, k, v, z, r, st, 32);   // zero-filled tile columns
    else return run<T, D, K>(p, k, v, z, r, st);
}

template <typename T, int D>
int by_k(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    switch (p.K) {
        case 1: return pick<T, D, 1>(p, k, v, z, r, st);
        case 3: return pick<T, D, 3>(p, k, v, z, r, st);
        case 5: return pick<T, D, 5>(p, k, v, z, r, st);
        case 7: return pick<T, D, 7>(p, k, v, z, r, st);
        case 9: return pick<T, D, 9>(p, k, v, z, r, st);
        case 11: return pick<T, D, 11>(p, k, v, z, r, st);
        case 13: return pick<T, D, 13>(p, k, v, z, r, st);
    }
    return LTE_ERR_UNSUPPORTED;
}

template <typename T>
int by_d(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    switch (p.d) {
        case 32: return by_k<T, 32>(p, k, v, z, r, st);
        case 64: return by_k<T, 64>(p, k, v, z, r, st);
        case 128: return by_k<T, 128>(p, k, v, z, r, st);
    }
    return LTE_ERR_UNSUPPORTED;
}

}  // namespace

int scores_status_fetch_and_clear() { return status_fetch_and_clear(g_scores_status); }

int launch_scores(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    return p.dtype == LTE_BF16 ? by_d<__nv_bfloat16>(p, k, v, z, r, st) : by_d<float>(p, k, v, z, r, st);
}

}  // namespace lte

#ifdef LTE_PROFILE
extern "C" int lte_sprof_read(long long* out)
{
    return cudaMemcpyFromSymbol(out, lte::g_sprof, sizeof(long long) * 64) == cudaSuccess ? 0 : -1;
}
#endif
