// Backward of the paper's scorer stack on the tcgen05 tensor cores (bf16 inputs, d = 64): the same quantities as the
// fp32 kernel in scores_stack_bwd.cu.  Gradients tolerate bf16 operands (fp32 accumulation), so nothing is split here.
//
// Row m of a tile of 128 rows is time tb + m, tb = a - 16; the tile owns the 96 times a .. a+95 (rows 16 .. 111); the
// rows before and after are the halo that the forward (12 earlier rows) and the transposed products (12 later rows)
// need.  Operands live in the unswizzled chunk-column layout of the forward kernel (a column of 16-byte chunks per 8
// channels, rows 16 bytes apart), which serves three kinds of product:
//   forward          D[t][o]  += in[t - shift][c] W[o][tau][c]     A = tile shifted in rows, K-major (K = c)
//   transposed       g[t][c]  += delta[t + shift][o] W[o][tau][c]  A = delta tile shifted in rows, K-major (K = o)
//   weight gradient  dW[c][o] += in[t - shift][c] delta[t][o]      A = in tile, B = delta tile, both MN-major (K = t, 16
//                                                                  rows per step, the tile's own rows only)
// The weight gradients of all three layers accumulate in tensor memory (336 columns) across the CTA's tiles.  Per tile the
// MMA warp and the eight epilogue warps alternate through six phases: forward x3 (epilogue: activation as the next
// operand, Swish' kept in registers), then per layer downwards the weight gradient together with the transposed
// product (epilogue: delta of the layer below = g Swish', as the next operand); the last transposed product is the
// input gradient, added to dk, dv.  Bias gradients and the output map's are per-thread sums in registers.
#include "tc_common.cuh"

namespace lte {

__device__ StatusWord g_stack_bwd_status = LTE_STATUS_INIT;

namespace {

using namespace tc;

constexpr int BT_ROWS = 136, BT_COL = BT_ROWS * 16;            // chunk column: 136 rows of 16 bytes
constexpr int BT_OWN0 = 16, BT_OWN = 96;                       // the tile's own rows
constexpr int BT_THREADS = 288;                                // 8 epilogue warps and the warp that issues the MMAs and the loads
// weight image per head (bf16, one piece): forward operands [tap][chunk of c_in][o][8], transposed [tap][chunk of o][c_in][8]
constexpr int BI_F0 = 3 * 16 * 64 * 16, BI_F1 = 3 * 8 * 32 * 16, BI_F2 = 3 * 4 * 16 * 16;
constexpr int BI_T0 = 3 * 8 * 128 * 16, BI_T1 = 3 * 4 * 64 * 16, BI_T2 = 3 * 2 * 32 * 16;
constexpr int BI_PAR = 640;                                    // floats: b0[64] b1[32] b2[16] wout[16] bout
constexpr int BI_HEAD = BI_F0 + BI_F1 + BI_F2 + BI_T0 + BI_T1 + BI_T2 + BI_PAR;   // 129,664
// shared memory
constexpr int BO_W = 0;                                        // the head's image
constexpr int BO_X = BO_W + BI_HEAD;                           // input tile: 16 columns (row rho = m + 4)
constexpr int BO_H0 = BO_X + 16 * BT_COL;                      // h0: 8 columns (row 8 + m), then a column of ones
constexpr int BO_H1 = BO_H0 + 9 * BT_COL;                      // h1: 4 columns (row 8 + m), then a column of ones
constexpr int BO_D0 = BO_H1 + 5 * BT_COL;                      // delta0: 8 columns (row m)
constexpr int BO_D1 = BO_D0 + 8 * BT_COL;                      // delta1: 4 columns
constexpr int BO_D2 = BO_D1 + 4 * BT_COL;                      // delta2: 2 columns
constexpr int BO_BAR = BO_D2 + 2 * BT_COL;
constexpr int BT_SMEM = BO_BAR + 64;
static_assert(BT_SMEM <= 232448 && (BO_X % 128) == 0, "shared memory");
// tensor memory columns
constexpr uint32_t TC_F = 0, TC_W0 = 128, TC_W1 = 320, TC_W2 = 416, BT_TMEM = 512;
constexpr uint32_t kFlatHi = (128u >> 4) | (1u << 14);         // unswizzled K-major: SBO = 128 (next 8 rows), LBO in the low word
// unswizzled MN-major: the 8 x 16-byte core matrices of one chunk column are 128 bytes apart along K (rows), the next 8
// channels are a chunk column further
constexpr uint32_t kMnHi = ((uint32_t)BT_COL >> 4) | (1u << 14);
__device__ __forceinline__ uint32_t mn_lo(uint32_t addr) { return (addr >> 4) | ((128u >> 4) << 16); }

// packed per-CTA partial gradient (same layout as the fp32 kernel's): wl0 [64][3][128] | wl1 [32][3][64] | wl2 [16][3][32] |
// wout [16] | b0 [64] | b1 [32] | b2 [16] | bout
constexpr int BG0 = 64 * 3 * 128, BG1 = 32 * 3 * 64, BG2 = 16 * 3 * 32;
constexpr int BPART = BG0 + BG1 + BG2 + 16 + 64 + 32 + 16 + 1, BPART_PAD = (BPART + 31) & ~31;

__device__ __forceinline__ void bwait(uint32_t bar, uint32_t parity, int code) {
    for (uint32_t i = 0; i < (1u << 20); ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
        if (ok) return;
        if ((i & 255u) == 255u && launch_aborted(&g_stack_bwd_status)) return;   // another wait of this launch has given up
    }
    wait_gave_up(&g_stack_bwd_status, code);
}
__device__ __forceinline__ void tmem_ld16b(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void st_chunk(uint32_t dst, const uint32_t (&wv)[4]) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(wv[0]), "r"(wv[1]), "r"(wv[2]), "r"(wv[3]) : "memory");
}

// ---- weight image: blockIdx.x = head ------------------------------------------------------------------------------
__global__ void stack_bwd_image_kernel(const float* __restrict__ wpack, const float* __restrict__ bpack, uint8_t* __restrict__ img, int H)
{
    pdl_launch_dependents();
    pdl_wait();
    const int h = blockIdx.x, tid = blockIdx.y * blockDim.x + threadIdx.x, nthr = gridDim.y * blockDim.x;
    uint8_t* out = img + (size_t)h * BI_HEAD;
    const float* g0 = wpack + (size_t)h * BG0;
    const float* g1 = wpack + (size_t)H * BG0 + (size_t)h * BG1;
    const float* g2 = wpack + (size_t)H * (BG0 + BG1) + (size_t)h * BG2;
    const float* go = wpack + (size_t)H * (BG0 + BG1 + BG2) + (size_t)h * 16;
    // g [o][tau][c]; forward image [tau][c / 8][o][c % 8], transposed image [tau][o / 8][c][o % 8]
    auto fill = [&](uint8_t* fdst, uint8_t* tdst, const float* g, int cin, int cout) {
        __nv_bfloat16* f = reinterpret_cast<__nv_bfloat16*>(fdst);
        __nv_bfloat16* t = reinterpret_cast<__nv_bfloat16*>(tdst);
        for (int e = tid; e < cout * 3 * cin; e += nthr) {
            const int c = e % cin, ot = e / cin, tau = ot % 3, o = ot / 3;
            const __nv_bfloat16 w = __float2bfloat16_rn(g[e]);
            f[((tau * (cin / 8) + c / 8) * cout + o) * 8 + (c & 7)] = w;
            t[((tau * (cout / 8) + o / 8) * cin + c) * 8 + (o & 7)] = w;
        }
    };
    fill(out, out + BI_F0 + BI_F1 + BI_F2, g0, 128, 64);
    fill(out + BI_F0, out + BI_F0 + BI_F1 + BI_F2 + BI_T0, g1, 64, 32);
    fill(out + BI_F0 + BI_F1, out + BI_F0 + BI_F1 + BI_F2 + BI_T0 + BI_T1, g2, 32, 16);
    float* par = reinterpret_cast<float*>(out + BI_HEAD - BI_PAR);
    for (int e = tid; e < BI_PAR / 4; e += nthr) {
        float x = 0.f;
        if (e < 64) x = bpack ? bpack[(size_t)h * 64 + e] : 0.f;
        else if (e < 96) x = bpack ? bpack[(size_t)H * 64 + (size_t)h * 32 + (e - 64)] : 0.f;
        else if (e < 112) x = bpack ? bpack[(size_t)H * 96 + (size_t)h * 16 + (e - 96)] : 0.f;
        else if (e < 128) x = go[e - 112];
        else if (e == 128) x = bpack ? bpack[(size_t)H * 112 + h] : 0.f;
        par[e] = x;
    }
}

// ---- main kernel: grid (chunks, B H), a CTA walks tiles of one (b,h) row ---------------------------------------------
__global__ void __launch_bounds__(BT_THREADS, 1)
stack_bwd_tc_kernel(const __nv_bfloat16* __restrict__ kg, const __nv_bfloat16* __restrict__ vg, const uint8_t* __restrict__ img,
                    const float* __restrict__ dz, __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                    float* __restrict__ part, int H, int Tlen, int tiles_per_cta, int input_grad)
{
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 127u) != 0) { if (threadIdx.x == 0) atomicExch(&g_stack_bwd_status.code, 9); return; }
    const uint32_t sW = base + BO_W, sX = base + BO_X, sH0 = base + BO_H0, sH1 = base + BO_H1;
    const uint32_t sD0 = base + BO_D0, sD1 = base + BO_D1, sD2 = base + BO_D2;
    const uint32_t sF0 = sW, sF1 = sF0 + BI_F0, sF2 = sF1 + BI_F1, sT0 = sF2 + BI_F2, sT1 = sT0 + BI_T0, sT2 = sT1 + BI_T1;
    const float* par = reinterpret_cast<const float*>(smem_raw + BO_W + BI_HEAD - BI_PAR);
    const uint32_t bar_w = base + BO_BAR, bar_x = bar_w + 8, bar_m = bar_w + 16, bar_e = bar_w + 24, tmem_slot = bar_w + 32;
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_raw + BO_BAR + 32);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.y, h = bh % H;
    const int n_tiles = (Tlen + BT_OWN - 1) / BT_OWN;
    const int tile_begin = blockIdx.x * tiles_per_cta, tile_end = min(tile_begin + tiles_per_cta, n_tiles);
    const int n_my = tile_end > tile_begin ? tile_end - tile_begin : 0;
    float* my_part = part + ((size_t)bh * gridDim.x + blockIdx.x) * BPART_PAD;

    // activation and delta columns start as zeros, the two extra columns as ones (bf16 1.0 = 0x3f80)
    for (int e = tid; e < (BO_BAR - BO_X) / 16; e += BT_THREADS) {
        const uint32_t off = BO_X + e * 16;
        const bool ones = (off >= BO_H0 + 8 * BT_COL && off < BO_H1) || (off >= BO_H1 + 4 * BT_COL && off < BO_D0);
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base + off), "r"(ones ? 0x3f803f80u : 0u) : "memory");
    }
    if (tid == 0) {
        mbar_init(bar_w, 1); mbar_init(bar_x, 1); mbar_init(bar_m, 1); mbar_init(bar_e, 8);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 8) tmem_alloc(tmem_slot, BT_TMEM);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;

    if (warp == 8) {
        // =================================== MMA issue and loads ===========================================
        const bool leader = lane == 0;
        if (leader && n_my > 0) {
            mbar_expect_tx(bar_w, BI_HEAD);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(sW), "l"(img + (size_t)h * BI_HEAD), "r"((uint32_t)BI_HEAD), "r"(bar_w) : "memory");
        }
        // input rows tb-4 .. tb+127 into their chunk columns (16-byte copies, rows outside [0, T) zero-filled)
        auto load_x = [&](int tile) {
            const __nv_bfloat16* kb = kg + (size_t)bh * Tlen * 64;
            const __nv_bfloat16* vb = vg + (size_t)bh * Tlen * 64;
            const int t0 = tile * BT_OWN - BT_OWN0 - 4, r_in = lane & 7, cq = lane >> 3;
#pragma unroll 1
            for (int rb = 0; rb < (132 + 7) / 8; ++rb) {
                const int r = rb * 8 + r_in, t = t0 + r;
                const bool ok = r < 132 && t >= 0 && t < Tlen;
                if (r < 132) {
#pragma unroll
                    for (int cg = 0; cg < 4; ++cg) {
                        const int c = cg * 4 + cq;
                        const __nv_bfloat16* src = (cg < 2 ? kb : vb) + (size_t)(ok ? t : 0) * 64 + (c & 7) * 8;
                        cp_async16(sX + c * BT_COL + r * 16, src, ok ? 16u : 0u);
                    }
                }
            }
            cp_async_commit();
            cp_async_wait<0>();
            fence_proxy_async();
            __syncwarp();
        };
        constexpr uint32_t ID_N64 = instr_desc(128, 64, false), ID_N32 = instr_desc(128, 32, false), ID_N16 = instr_desc(128, 16, false);
        constexpr uint32_t ID_N128 = instr_desc(128, 128, false);
        constexpr uint32_t IW_N64 = instr_desc(128, 64, true, true), IW_N32 = instr_desc(128, 32, true, true), IW_N16 = instr_desc(128, 16, true, true);
        // K-major operand: chunk column pair of a K step, LBO = distance between the two columns
        auto kdesc = [](uint32_t addr, uint32_t lbo) { return desc64(desc_lo(addr, lbo), kFlatHi); };
        auto mdesc = [](uint32_t addr) { return desc64(mn_lo(addr), kMnHi); };
        if (n_my > 0) { load_x(tile_begin); bwait(bar_w, 0, 1); }
        for (int it = 0; it < n_my; ++it) {
            const uint32_t ph = 6u * (uint32_t)it;
            tc_fence_after();
            // ---- M1: layer 0 forward ----
            if (leader) {
#pragma unroll
                for (int tau = 0; tau < 3; ++tau)
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        umma(tmem + TC_F, kdesc(sX + 2 * kk * BT_COL + 2 * tau * 16, BT_COL),
                             kdesc(sF0 + (tau * 16 + 2 * kk) * 64 * 16, 64 * 16), ID_N64, (tau > 0 || kk > 0) ? 1u : 0u);
                umma_commit(bar_m);
            }
            __syncwarp();
            bwait(bar_e, (ph + 0) & 1, 2);
            tc_fence_after();
            // ---- M2: layer 1 forward ----
            if (leader) {
#pragma unroll
                for (int tau = 0; tau < 3; ++tau)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma(tmem + TC_F, kdesc(sH0 + 2 * kk * BT_COL + (4 + 2 * tau) * 16, BT_COL),
                             kdesc(sF1 + (tau * 8 + 2 * kk) * 32 * 16, 32 * 16), ID_N32, (tau > 0 || kk > 0) ? 1u : 0u);
                umma_commit(bar_m);
            }
            __syncwarp();
            bwait(bar_e, (ph + 1) & 1, 3);
            tc_fence_after();
            // ---- M3: layer 2 forward ----
            if (leader) {
#pragma unroll
                for (int tau = 0; tau < 3; ++tau)
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk)
                        umma(tmem + TC_F, kdesc(sH1 + 2 * kk * BT_COL + (4 + 2 * tau) * 16, BT_COL),
                             kdesc(sF2 + (tau * 4 + 2 * kk) * 16 * 16, 16 * 16), ID_N16, (tau > 0 || kk > 0) ? 1u : 0u);
                umma_commit(bar_m);
            }
            __syncwarp();
            bwait(bar_e, (ph + 2) & 1, 4);
            tc_fence_after();
            // ---- M4: layer 2 weight gradient (in = h1 with its ones column: lane 32 collects the bias gradient) and
            // the transposed product towards layer 1 ----
            if (leader) {
#pragma unroll
                for (int tau = 0; tau < 3; ++tau)
#pragma unroll
                    for (int ks = 0; ks < BT_OWN / 16; ++ks)
                        umma(tmem + TC_W2 + tau * 16, mdesc(sH1 + (8 + BT_OWN0 - 4 + 2 * tau + 16 * ks) * 16),
                             mdesc(sD2 + (BT_OWN0 + 16 * ks) * 16), IW_N16, (it > 0 || ks > 0) ? 1u : 0u);
#pragma unroll
                for (int tp = 0; tp < 3; ++tp)
                    umma(tmem + TC_F, kdesc(sD2 + 2 * tp * 16, BT_COL), kdesc(sT2 + ((2 - tp) * 2) * 32 * 16, 32 * 16), ID_N32, tp > 0 ? 1u : 0u);
                umma_commit(bar_m);
            }
            __syncwarp();
            bwait(bar_e, (ph + 3) & 1, 5);
            tc_fence_after();
            // ---- M5: layer 1 weight gradient (lane 64: bias gradient) and the transposed product towards layer 0 ----
            if (leader) {
#pragma unroll
                for (int tau = 0; tau < 3; ++tau)
#pragma unroll
                    for (int ks = 0; ks < BT_OWN / 16; ++ks)
                        umma(tmem + TC_W1 + tau * 32, mdesc(sH0 + (8 + BT_OWN0 - 4 + 2 * tau + 16 * ks) * 16),
                             mdesc(sD1 + (BT_OWN0 + 16 * ks) * 16), IW_N32, (it > 0 || ks > 0) ? 1u : 0u);
#pragma unroll
                for (int tp = 0; tp < 3; ++tp)
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk)
                        umma(tmem + TC_F, kdesc(sD1 + 2 * kk * BT_COL + 2 * tp * 16, BT_COL),
                             kdesc(sT1 + ((2 - tp) * 4 + 2 * kk) * 64 * 16, 64 * 16), ID_N64, (tp > 0 || kk > 0) ? 1u : 0u);
                umma_commit(bar_m);
            }
            __syncwarp();
            bwait(bar_e, (ph + 4) & 1, 6);
            tc_fence_after();
            // ---- M6: layer 0 weight gradient and the input gradient ----
            if (leader) {
#pragma unroll
                for (int tau = 0; tau < 3; ++tau)
#pragma unroll
                    for (int ks = 0; ks < BT_OWN / 16; ++ks)
                        umma(tmem + TC_W0 + tau * 64, mdesc(sX + (4 + BT_OWN0 - 4 + 2 * tau + 16 * ks) * 16),
                             mdesc(sD0 + (BT_OWN0 + 16 * ks) * 16), IW_N64, (it > 0 || ks > 0) ? 1u : 0u);
                if (input_grad) {
#pragma unroll
                    for (int tp = 0; tp < 3; ++tp)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma(tmem + TC_F, kdesc(sD0 + 2 * kk * BT_COL + 2 * tp * 16, BT_COL),
                                 kdesc(sT0 + ((2 - tp) * 8 + 2 * kk) * 128 * 16, 128 * 16), ID_N128, (tp > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(bar_m);
            }
            __syncwarp();
            // the input tile is free once these products have completed: this warp watches the same barrier as the epilogue
            bwait(bar_m, (ph + 5) & 1, 7);
            if (it + 1 < n_my) load_x(tile_begin + it + 1);
            bwait(bar_e, (ph + 5) & 1, 8);
        }
        // ---- weight gradients out of tensor memory: done by the epilogue warps below after this barrier ----
    }
    else {
        // =================================== epilogue warps ================================================
        // warp w owns TMEM lanes 32 (w & 3) .. +31 (row m) and half (w >> 2) of a layer's channels
        const int q = warp & 3, half = warp >> 2;
        const int m = q * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(q * 32)) << 16;
        const bool own = m >= BT_OWN0 && m < BT_OWN0 + BT_OWN;
        auto f = [](uint32_t u) { return __uint_as_float(u); };
        float sp0[32], sp1[16], sp2[8];                        // Swish' of this thread's positions, kept from the forward phases
        float db0[32], dwo[8], dbo = 0.f;                      // sums over the own rows of all tiles (bias 0, output map)
#pragma unroll
        for (int c = 0; c < 32; ++c) db0[c] = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) dwo[c] = 0.f;
        auto phase_done = [&]() {
            fence_proxy_async();                               // what this phase stored is an MMA operand of the next one
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_e);
        };
        if (n_my > 0) bwait(bar_w, 0, 10);
        for (int it = 0; it < n_my; ++it) {
            const uint32_t ph = 6u * (uint32_t)it;
            const int time = (tile_begin + it) * BT_OWN - BT_OWN0 + m;
            const float live = time >= 0 ? 1.f : 0.f;          // every layer's output is zero at negative times
            const float d3 = (time >= 6 && time < Tlen) ? dz[(size_t)bh * Tlen + time - 6] : 0.f;   // dL/d(output at this time)
            // ---- E1: h0 and Swish'(y0), 32 channels ----
            bwait(bar_m, (ph + 0) & 1, 11);
            tc_fence_after();
            {
                uint32_t a[32];
                tmem_ld32(tmem + lane_base + TC_F + half * 32, a);
                tmem_wait_ld();
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t wv[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float hv[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int c = ch * 8 + 2 * e + u;
                            const float y = f(a[c]) + par[half * 32 + c];
                            const float sg = __fdividef(1.f, 1.f + __expf(-y));
                            hv[u] = live * y * sg;
                            sp0[c] = live * sg * (1.f + y * (1.f - sg));
                        }
                        wv[e] = pack2(hv[0], hv[1]);
                    }
                    st_chunk(sH0 + (uint32_t)(half * 4 + ch) * BT_COL + (uint32_t)(8 + m) * 16, wv);
                }
            }
            phase_done();
            // ---- E2: h1 and Swish'(y1), 16 channels ----
            bwait(bar_m, (ph + 1) & 1, 12);
            tc_fence_after();
            {
                uint32_t a[16];
                tmem_ld16b(tmem + lane_base + TC_F + half * 16, a);
                tmem_wait_ld();
#pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    uint32_t wv[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float hv[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int c = ch * 8 + 2 * e + u;
                            const float y = f(a[c]) + par[64 + half * 16 + c];
                            const float sg = __fdividef(1.f, 1.f + __expf(-y));
                            hv[u] = live * y * sg;
                            sp1[c] = live * sg * (1.f + y * (1.f - sg));
                        }
                        wv[e] = pack2(hv[0], hv[1]);
                    }
                    st_chunk(sH1 + (uint32_t)(half * 2 + ch) * BT_COL + (uint32_t)(8 + m) * 16, wv);
                }
            }
            phase_done();
            // ---- E3: h2 (8 channels per thread), the output map's gradient, delta2 = d3 wout Swish'(y2) ----
            bwait(bar_m, (ph + 2) & 1, 13);
            tc_fence_after();
            {
                uint32_t a[16];
                tmem_ld16b(tmem + lane_base + TC_F + half * 8, a);   // this thread's 8 channels are the first 8 loaded
                tmem_wait_ld();
                uint32_t wv[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float dv2[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int c = 2 * e + u, cc = half * 8 + c;
                        const float y = f(a[c]) + par[96 + cc];
                        const float sg = __fdividef(1.f, 1.f + __expf(-y));
                        const float h2 = live * y * sg;
                        sp2[c] = live * sg * (1.f + y * (1.f - sg));
                        if (own) dwo[c] = fmaf(d3, h2, dwo[c]);
                        dv2[u] = d3 * par[112 + cc] * sp2[c];
                    }
                    wv[e] = pack2(dv2[0], dv2[1]);
                }
                st_chunk(sD2 + (uint32_t)half * BT_COL + (uint32_t)m * 16, wv);
                if (own && half == 0) dbo += d3;
            }
            phase_done();
            // ---- E4: delta1 = g1 Swish'(y1) ----
            bwait(bar_m, (ph + 3) & 1, 14);
            tc_fence_after();
            {
                uint32_t a[16];
                tmem_ld16b(tmem + lane_base + TC_F + half * 16, a);
                tmem_wait_ld();
#pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    uint32_t wv[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int c = ch * 8 + 2 * e;
                        wv[e] = pack2(f(a[c]) * sp1[c], f(a[c + 1]) * sp1[c + 1]);
                    }
                    st_chunk(sD1 + (uint32_t)(half * 2 + ch) * BT_COL + (uint32_t)m * 16, wv);
                }
            }
            phase_done();
            // ---- E5: delta0 = g0 Swish'(y0); bias gradient of layer 0 in registers (its weight gradient has no spare lane) ----
            bwait(bar_m, (ph + 4) & 1, 15);
            tc_fence_after();
            {
                uint32_t a[32];
                tmem_ld32(tmem + lane_base + TC_F + half * 32, a);
                tmem_wait_ld();
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t wv[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int c = ch * 8 + 2 * e;
                        const float d0a = f(a[c]) * sp0[c], d0b = f(a[c + 1]) * sp0[c + 1];
                        if (own) { db0[c] += d0a; db0[c + 1] += d0b; }
                        wv[e] = pack2(d0a, d0b);
                    }
                    st_chunk(sD0 + (uint32_t)(half * 4 + ch) * BT_COL + (uint32_t)m * 16, wv);
                }
            }
            phase_done();
            // ---- E6: the input gradient of the own rows, added to dk (first 64 channels) / dv (the other 64) ----
            bwait(bar_m, (ph + 5) & 1, 16);
            tc_fence_after();
            if (input_grad) {
                __nv_bfloat16* dst = (half == 0 ? dk : dv) + ((size_t)bh * Tlen + (time >= 0 && time < Tlen ? time : 0)) * 64;
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
                    uint32_t a[32];
                    tmem_ld32(tmem + lane_base + TC_F + half * 64 + cb * 32, a);
                    tmem_wait_ld();
                    if (own && time < Tlen) {
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {
                            uint4* p4 = reinterpret_cast<uint4*>(dst + cb * 32 + ch * 8);
                            const uint4 old = *p4;
                            const uint32_t ow[4] = {old.x, old.y, old.z, old.w};
                            uint32_t nw[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                nw[e] = pack2(__uint_as_float(ow[e] << 16) + f(a[ch * 8 + 2 * e]),
                                              __uint_as_float(ow[e] & 0xffff0000u) + f(a[ch * 8 + 2 * e + 1]));
                            *p4 = make_uint4(nw[0], nw[1], nw[2], nw[3]);
                        }
                    }
                }
            }
            phase_done();
        }
        // ---- per-thread sums -> shared memory (the operand buffers are free now) -> fixed-order column sums ----
        __syncwarp();
        asm volatile("bar.sync 1, 256;" ::: "memory");         // every epilogue warp is past its last phase
        float* red = reinterpret_cast<float*>(smem_raw + BO_X);   // [128 rows][64 + 16 + 1]: b0 | wout | bout
        {
            float* row = red + (size_t)m * 81;
#pragma unroll
            for (int c = 0; c < 32; ++c) row[half * 32 + c] = db0[c];
#pragma unroll
            for (int c = 0; c < 8; ++c) row[64 + half * 8 + c] = dwo[c];
            if (half == 0) row[80] = dbo;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (tid < 81) {
            float t = 0.f;
            for (int r = 0; r < 128; ++r) t += red[(size_t)r * 81 + tid];
            float* sp = my_part + BG0 + BG1 + BG2;             // wout [16] | b0 [64] | b1 [32] | b2 [16] | bout
            if (tid < 64) sp[16 + tid] = t;
            else if (tid < 80) sp[tid - 64] = t;
            else sp[16 + 112] = t;
        }
    }
    // ---- weight gradients out of tensor memory (lane = input channel), bias gradients of layers 1 and 2 from the ones lanes ----
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp < 4) {
        const int c = warp * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;
        float* sp = my_part + BG0 + BG1 + BG2;
        for (int cb = 0; cb < 6; ++cb) {                       // layer 0: 3 taps x 64 outputs
            uint32_t a[32];
            if (n_my > 0) { tmem_ld32(tmem + lane_base + TC_W0 + cb * 32, a); tmem_wait_ld(); }
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                const int col = cb * 32 + e, tau = col / 64, o = col % 64;
                my_part[(o * 3 + tau) * 128 + c] = n_my > 0 ? __uint_as_float(a[e]) : 0.f;
            }
        }
        for (int cb = 0; cb < 3; ++cb) {                       // layer 1: 3 taps x 32 outputs, lanes 0..63; lane 64: bias gradient
            uint32_t a[32];
            if (n_my > 0) { tmem_ld32(tmem + lane_base + TC_W1 + cb * 32, a); tmem_wait_ld(); }
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                const float x = n_my > 0 ? __uint_as_float(a[e]) : 0.f;
                if (c < 64) my_part[BG0 + (e * 3 + cb) * 64 + c] = x;
                else if (c == 64 && cb == 0) sp[16 + 64 + e] = x;
            }
        }
        for (int cb = 0; cb < 3; ++cb) {                       // layer 2: 3 taps x 16 outputs, lanes 0..31; lane 32: bias gradient
            uint32_t a[16];
            if (n_my > 0) { tmem_ld16b(tmem + lane_base + TC_W2 + cb * 16, a); tmem_wait_ld(); }
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const float x = n_my > 0 ? __uint_as_float(a[e]) : 0.f;
                if (c < 32) my_part[BG0 + BG1 + (e * 3 + cb) * 32 + c] = x;
                else if (c == 32 && cb == 0) sp[16 + 96 + e] = x;
            }
        }
    }
    if (n_my == 0 && threadIdx.x < 81) {                       // a CTA without tiles contributes zeros
        float* sp = my_part + BG0 + BG1 + BG2;
        if (threadIdx.x < 64) sp[16 + threadIdx.x] = 0.f; else if (threadIdx.x < 80) sp[threadIdx.x - 64] = 0.f; else sp[128] = 0.f;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, BT_TMEM);
}

// the same fixed-order sum of the CTAs' partials as the fp32 kernel's
__global__ void stack_bwd_tc_reduce_kernel(const float* __restrict__ part, float* __restrict__ dw, float* __restrict__ dbias,
                                           int B, int H, int chunks)
{
    pdl_launch_dependents();
    pdl_wait();
    const int h = blockIdx.y, e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= BPART) return;
    float t = 0.f;
    for (int b = 0; b < B; ++b)
        for (int ch = 0; ch < chunks; ++ch) t += part[(((size_t)b * H + h) * chunks + ch) * BPART_PAD + e];
    if (e < BG0) dw[(size_t)h * BG0 + e] = t;
    else if (e < BG0 + BG1) dw[(size_t)H * BG0 + (size_t)h * BG1 + (e - BG0)] = t;
    else if (e < BG0 + BG1 + BG2) dw[(size_t)H * (BG0 + BG1) + (size_t)h * BG2 + (e - BG0 - BG1)] = t;
    else if (e < BG0 + BG1 + BG2 + 16) dw[(size_t)H * (BG0 + BG1 + BG2) + (size_t)h * 16 + (e - BG0 - BG1 - BG2)] = t;
    else if (dbias) {
        const int f = e - (BG0 + BG1 + BG2 + 16);
        if (f < 64) dbias[(size_t)h * 64 + f] = t;
        else if (f < 96) dbias[(size_t)H * 64 + (size_t)h * 32 + (f - 64)] = t;
        else if (f < 112) dbias[(size_t)H * 96 + (size_t)h * 16 + (f - 96)] = t;
        else dbias[(size_t)H * 112 + h] = t;
    }
}

int bt_chunks(const Params& p)
{
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int BH = p.B * p.H, n_tiles = (p.T + BT_OWN - 1) / BT_OWN;
    // row chunks per (b,h): the split that minimises waves x (tiles per CTA + about one tile of set-up and write-out)
    int best = 1;
    long best_cost = -1;
    for (int chunks = 1; chunks <= n_tiles && chunks <= 64; ++chunks) {
        const int per = (n_tiles + chunks - 1) / chunks, eff = (n_tiles + per - 1) / per;
        const long waves = ((long)BH * eff + sms - 1) / sms, cost = waves * (per + 1);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = eff; }
    }
    return best;
}

}  // namespace

int stack_bwd_tc_status_fetch_and_clear() { return status_fetch_and_clear(g_stack_bwd_status); }

// scratch: the weight image, then one packed partial gradient per CTA; 0 where the tensor-core path does not apply
size_t stack_bwd_tc_workspace(const Params& p)
{
    if (p.dtype != LTE_BF16 || p.d != 64) return 0;
    return ((size_t)p.H * BI_HEAD + 255) / 256 * 256 + (size_t)p.B * p.H * bt_chunks(p) * BPART_PAD * sizeof(float);
}

int launch_stack_bwd_tc(const Params& p, const void* k, const void* v, const float* dz, void* dk, void* dv, float* dw,
                        float* dbias, bool input_grad, void* ws, cudaStream_t st)
{
    if (p.dtype != LTE_BF16 || p.d != 64) return LTE_ERR_UNSUPPORTED;
    static PerDeviceOnce attr;
    if (int e = attr.run([] { return cudaFuncSetAttribute(stack_bwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, BT_SMEM); })) return e;
    uint8_t* img = (uint8_t*)ws;
    float* part = (float*)((char*)ws + ((size_t)p.H * BI_HEAD + 255) / 256 * 256);
    if (launch_pdl(stack_bwd_image_kernel, dim3(p.H, 32), dim3(256), 0, st, p.w, p.bias, img, p.H) != cudaSuccess) return LTE_ERR_CUDA;
    const int chunks = bt_chunks(p);
    const int n_tiles = (p.T + BT_OWN - 1) / BT_OWN, per = (n_tiles + chunks - 1) / chunks;
    if (launch_pdl(stack_bwd_tc_kernel, dim3(chunks, p.B * p.H), dim3(BT_THREADS), BT_SMEM, st, (const __nv_bfloat16*)k,
                   (const __nv_bfloat16*)v, (const uint8_t*)img, dz, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, part, p.H, p.T, per,
                   input_grad ? 1 : 0) != cudaSuccess)
        return LTE_ERR_CUDA;
    if (launch_pdl(stack_bwd_tc_reduce_kernel, dim3((BPART + 255) / 256, p.H), dim3(256), 0, st, (const float*)part, dw, dbias,
                   p.B, p.H, chunks) != cudaSuccess)
        return LTE_ERR_CUDA;
    return cuda_status(cudaGetLastError());
}

}  // namespace lte
