// The paper's scorer stack on the tcgen05 tensor cores (Section 3.1.1, hyper-parameters of Appendix A), bf16 inputs,
// d = 64: three dilated conv layers (kernel 3, dilation 2) over x = [k ; v], channels 128 -> 64 -> 32 -> 16, Swish
// after each, then a per-head linear map to one logit; the logit of token j is the stack's output at time j + 6.
//
// The keep decision z > logit(tau) has to agree with an fp64 evaluation to a few 1e-5 on z, so every product is
// exact: fp32 weights and fp32 hidden activations are split into three bf16 pieces (hi + mid + lo, 24 bits), and the
// pieces whose product matters (orders hi*hi, hi*mid, mid*hi, mid*mid, hi*lo, lo*hi) are accumulated in fp32 by the
// tensor core.  The pieces of a weight sit side by side along N (one MMA of N = 3 C_out covers hi, mid and lo at
// once; the epilogue adds the three column blocks), so an input tile is read from shared memory once per K step.
//
// A layer is a sum over its three taps of a [128 rows x C_in] x [C_in x C_out] product whose A operand is the
// previous layer's tile shifted down by 4, 2 or 0 rows.  Operands are kept in the unswizzled canonical layout (a
// column of 16-byte chunks per 8 channels, rows 16 bytes apart), where a row shift is a 16-byte-aligned change of the
// start address.  Row m of a tile is time tb - 8 + m: the input tile carries 4 more rows above, the first 4 rows of
// the second layer and the first 8 of the third are not used, so a tile yields 120 logits.
//
// One CTA per SM walks consecutive tiles of (head, batch) rows.  Warp 9 feeds shared memory: the input rows by
// 16-byte asynchronous copies into their chunk columns (rows before time 0 zero-filled), the first layer's weights tap by
// tap through a two-slot ring (their split image, 144 KB per head, does not fit beside the rest), the small layers'
// weights once per head.  Warp 8 issues the MMAs.  Warps 0-7 are the epilogues: TMEM -> bias, Swish -> three bf16
// pieces -> the next layer's operand in shared memory; the last one takes the dot product with the output vector.
// The weight image is built by a small kernel per call into caller-provided workspace.
#include "tc_common.cuh"

namespace lte {

__device__ StatusWord g_stack_tc_status = LTE_STATUS_INIT;
#ifdef LTE_PROFILE
__device__ long long g_stprof[64];
#define STP(i) do { if (blockIdx.x == 3 && it == 5 && lane == 0) g_stprof[i] = clock64(); } while (0)
#else
#define STP(i) do {} while (0)
#endif

namespace {

using namespace tc;

constexpr int ST_D = 64, ST_C0 = 128, ST_C1 = 64, ST_C2 = 32, ST_C3 = 16;
constexpr int ST_ROWS = 136;                                   // rows of a chunk column (132 input rows; 8 + 128 hidden rows)
constexpr int ST_COL = ST_ROWS * 16;                           // bytes of a chunk column
constexpr int ST_XROWS = 132;                                  // input rows per tile: times tb-12 .. tb+119
constexpr int ST_VALID = 120;                                  // logits per tile
constexpr int ST_HALF = 6;
constexpr int ST_THREADS = 352;                                // 8 epilogue warps, first-layer MMA warp, producer, later-layers MMA warp

// per-head image in the workspace (bytes): first-layer weights per tap, then what stays resident for the head
constexpr int IMG_W0_TAP = 16 * 192 * 16;                      // [chunk 16][n = piece * 64 + c_out][8 channels] bf16
constexpr int IMG_W0 = 3 * IMG_W0_TAP;
constexpr int IMG_W1 = 3 * 8 * 96 * 16;                        // [tap][chunk 8][n = piece * 32 + c_out][8]
constexpr int IMG_W2 = 3 * 4 * 48 * 16;                        // [tap][chunk 4][n = piece * 16 + c_out][8]
constexpr int IMG_PAR = 640;                                   // floats: b0[64] b1[32] b2[16] wout[16] bout
constexpr int IMG_RES = IMG_W1 + IMG_W2 + IMG_PAR;             // resident part, one bulk copy
constexpr int IMG_HEAD = IMG_W0 + IMG_RES;

// shared memory map (every offset a multiple of 128)
constexpr int OFF_RING = 0;                                    // 2 slots of IMG_W0_TAP
constexpr int OFF_X = OFF_RING + 2 * IMG_W0_TAP;               // input tile: 16 chunk columns
constexpr int OFF_HID = OFF_X + 16 * ST_COL;                   // 3 x 8 columns of h0; once the second layer has read them, the 3 x 4 of h1
constexpr int OFF_W1 = OFF_HID + 24 * ST_COL;
constexpr int OFF_W2 = OFF_W1 + IMG_W1;
constexpr int OFF_PAR = OFF_W2 + IMG_W2;
constexpr int OFF_BAR = OFF_PAR + IMG_PAR;
constexpr int ST_SMEM = OFF_BAR + 192;
static_assert(ST_SMEM <= 232448, "shared memory");
constexpr uint32_t D0_COL = 0, D1_COL = 384, D2_COL = 384, ST_TMEM = 512;   // two first-layer accumulators; the third layer's takes the second's columns

// unswizzled K-major descriptor: 8 rows x 16 bytes per core matrix, SBO = 128 bytes between 8-row groups, LBO = the
// distance between the two 8-channel chunk columns of a K = 16 step
constexpr uint32_t kDescHiFlat = (128u >> 4) | (1u << 14);

// Bounded wait.  The phases of this kernel are long (thousands of cycles) and at any time most warps are waiting, so the
// wait must not poll: try_wait is given a suspend-time hint and the thread sleeps in hardware until the phase
// completes (polling warps kept the shared-memory pipeline busy and slowed the working warps several times over).
__device__ __forceinline__ void swait(uint32_t bar, uint32_t parity, int code) {
    for (uint32_t i = 0; i < (1u << 20); ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
        if (ok) return;
        if ((i & 255u) == 255u && launch_aborted(&g_stack_tc_status)) return;   // another wait of this launch has given up
    }
    wait_gave_up(&g_stack_tc_status, code);
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
}
// Swish with the fast exponential and division: their error (a few 1e-7 relative) is below that of the tensor core's
// fp32 accumulation, which bounds the accuracy of the logits here (about 1e-5 absolute at |z| of a few units)
__device__ __forceinline__ float swish(float y) { return __fdividef(y, 1.f + __expf(-y)); }

// three bf16 pieces of two floats, packed (low half = a)
__device__ __forceinline__ void split3(float a, float b, uint32_t& hi, uint32_t& mid, uint32_t& lo) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    hi = *reinterpret_cast<uint32_t*>(&h);
    a -= __uint_as_float(hi << 16); b -= __uint_as_float(hi & 0xffff0000u);
    h = __floats2bfloat162_rn(a, b);
    mid = *reinterpret_cast<uint32_t*>(&h);
    a -= __uint_as_float(mid << 16); b -= __uint_as_float(mid & 0xffff0000u);
    h = __floats2bfloat162_rn(a, b);
    lo = *reinterpret_cast<uint32_t*>(&h);
}

// ---- weight image -------------------------------------------------------------------------------------------------
// blockIdx.x = head, the blocks along y share its elements.  wpack = wl0 | wl1 | wl2 | wout with wl[l] [H][c_out][3][c_in]; bpack = bl0 | bl1 | bl2 | bout or null.
// dg = the head dimension of the data, 64 or 32.  d = 32 runs the d = 64 kernel on a padded problem: channels [dg, 64) of the
// key and value halves of the input, and the upper half of every hidden layer, carry zero weights (and zero biases, so the
// padded activations are Swish(0) = 0); the image below is the d = 64 layout with those zeros written in.
__global__ void stack_image_kernel(const float* __restrict__ wpack, const float* __restrict__ bpack, uint8_t* __restrict__ img, int H, int dg)
{
    pdl_launch_dependents();
    pdl_wait();
    const int h = blockIdx.x, tid = blockIdx.y * blockDim.x + threadIdx.x, nthr = gridDim.y * blockDim.x;
    uint8_t* out = img + (size_t)h * IMG_HEAD;
    const int c0 = 2 * dg, c1 = dg, c2 = dg / 2, c3 = dg / 4;   // the real channel plan
    const float* g0 = wpack + (size_t)h * c1 * 3 * c0;
    const float* g1 = wpack + (size_t)H * c1 * 3 * c0 + (size_t)h * c2 * 3 * c1;
    const float* g2 = wpack + (size_t)H * (c1 * 3 * c0 + c2 * 3 * c1) + (size_t)h * c3 * 3 * c2;
    const float* go = wpack + (size_t)H * (c1 * 3 * c0 + c2 * 3 * c1 + c3 * 3 * c2) + (size_t)h * c3;
    auto piece = [](float w, int s) -> __nv_bfloat16 {
        __nv_bfloat16 p = __float2bfloat16_rn(w);
        for (int i = 0; i < s; ++i) { w -= __bfloat162float(p); p = __float2bfloat16_rn(w); }
        return p;
    };
    // padded dims cin x cout, real dims cin_r x cout_r; split: the input channels are two halves (key, value), each with its
    // real channels first
    auto fill = [&](uint8_t* dst, const float* g, int cin, int cout, int cin_r, int cout_r, bool split) {
        // dst [tap][chunk cin/8][n = piece * cout + o][8] ; g [o][tap][cin_r]
        const int n_el = 3 * cin * 3 * cout;
        __nv_bfloat16* d = reinterpret_cast<__nv_bfloat16*>(dst);
        for (int e = tid; e < n_el; e += nthr) {
            const int k8 = e & 7, n = (e >> 3) % (3 * cout), rest = (e >> 3) / (3 * cout), c = rest % (cin / 8), tau = rest / (cin / 8);
            const int s = n / cout, o = n % cout, ch = c * 8 + k8;
            int cr;
            if (split) { const int half = cin / 2, hr = cin_r / 2; cr = ch % half < hr ? (ch / half) * hr + ch % half : -1; }
            else cr = ch < cin_r ? ch : -1;
            d[e] = (o < cout_r && cr >= 0) ? piece(g[((size_t)o * 3 + tau) * cin_r + cr], s) : __float2bfloat16_rn(0.f);
        }
    };
    fill(out, g0, ST_C0, ST_C1, c0, c1, true);
    fill(out + IMG_W0, g1, ST_C1, ST_C2, c1, c2, false);
    fill(out + IMG_W0 + IMG_W1, g2, ST_C2, ST_C3, c2, c3, false);
    float* par = reinterpret_cast<float*>(out + IMG_W0 + IMG_W1 + IMG_W2);
    for (int e = tid; e < IMG_PAR / 4; e += nthr) {
        float x = 0.f;
        if (e < 64) x = (bpack && e < c1) ? bpack[(size_t)h * c1 + e] : 0.f;
        else if (e < 96) x = (bpack && e - 64 < c2) ? bpack[(size_t)H * c1 + (size_t)h * c2 + (e - 64)] : 0.f;
        else if (e < 112) x = (bpack && e - 96 < c3) ? bpack[(size_t)H * (c1 + c2) + (size_t)h * c3 + (e - 96)] : 0.f;
        else if (e < 128) x = e - 112 < c3 ? go[e - 112] : 0.f;
        else if (e == 128) x = bpack ? bpack[(size_t)H * (c1 + c2 + c3) + h] : 0.f;
        par[e] = x;
    }
}

// ---- main kernel --------------------------------------------------------------------------------------------------
struct StackWork { int h, bh, tb; };
__device__ __forceinline__ StackWork stack_work(int f, int n_t, int B, int H) {
    const int hb = f / n_t, tile = f - hb * n_t, h = hb / B, b = hb - h * B;
    return StackWork{h, b * H + h, ST_HALF + tile * ST_VALID};
}

__global__ void __launch_bounds__(ST_THREADS, 1)
scores_stack_tc_kernel(const __nv_bfloat16* __restrict__ kg, const __nv_bfloat16* __restrict__ vg,
                       const uint8_t* __restrict__ img, float* __restrict__ z, float* __restrict__ r_out, int B, int H,
                       int Tlen, int n_t, int n_flat, int per_cta, int dg)
{
    pdl_launch_dependents();
    pdl_wait();                                                // the weight image is written by the preceding kernel
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 127u) != 0) { if (threadIdx.x == 0) atomicExch(&g_stack_tc_status.code, 9); return; }
    const uint32_t sRing = base + OFF_RING, sX = base + OFF_X, sH0 = base + OFF_HID, sH1 = base + OFF_HID, sW1 = base + OFF_W1, sW2 = base + OFF_W2;
    const float* par = reinterpret_cast<const float*>(smem_raw + OFF_PAR);
    const uint32_t bar0 = base + OFF_BAR;
    const uint32_t bar_x = bar0, bar_rf = bar0 + 8, bar_re = bar0 + 24, bar_d0 = bar0 + 40, bar_d1 = bar0 + 48, bar_d2 = bar0 + 56;
    const uint32_t bar_h0 = bar0 + 64, bar_h1 = bar0 + 72, bar_w = bar0 + 88, bar_d0b = bar0 + 96, bar_f0 = bar0 + 104;
    const uint32_t bar_ed4 = bar0 + 128;                       // four barriers, one per tile modulo 4 (see the producer)
    const uint32_t tmem_slot = bar0 + 120;
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_raw + OFF_BAR + 120);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int f_begin = blockIdx.x * per_cta, f_end = min(f_begin + per_cta, n_flat);
    const int n_my = f_end - f_begin;

    // hidden-activation columns start out as zeros (their first rows are read by shifted operands before anything
    // meaningful is written there; what those rows produce is never used, but it should be finite)
    for (int e = tid; e < (24 * ST_COL) / 16; e += ST_THREADS)
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(sH0 + e * 16), "r"(0u) : "memory");
    if (tid == 0) {
        mbar_init(bar_x, 1);
        mbar_init(bar_rf, 1); mbar_init(bar_rf + 8, 1); mbar_init(bar_re, 1); mbar_init(bar_re + 8, 1);
        mbar_init(bar_d0, 1); mbar_init(bar_d0b, 1); mbar_init(bar_d1, 1); mbar_init(bar_d2, 1);
        mbar_init(bar_f0, 8); mbar_init(bar_f0 + 8, 8);
        mbar_init(bar_h0, 8); mbar_init(bar_h1, 8); mbar_init(bar_w, 1);
#pragma unroll
        for (int e = 0; e < 4; ++e) mbar_init(bar_ed4 + 8 * e, 4);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 8) tmem_alloc(tmem_slot, ST_TMEM);
    fence_proxy_async();                                       // the zero fill is visible to the TMA writes and MMA reads that follow
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;

    if (warp == 9) {
        // =================================== producer ======================================================
        const bool leader = lane == 0;
        // input rows tb-12 .. tb+119 into their chunk columns, 16 bytes per copy: a lane takes row (l & 7) of a block of 8
        // rows and one of 4 chunks, so a quarter warp writes 128 contiguous bytes and reads full 32-byte sectors.  Rows
        // outside [0, T) are zero-filled.  (Tensor-map copies with 16-byte boxes needed about 3,600 cycles per tile.)
        auto load_x = [&](const StackWork& w) {
            const __nv_bfloat16* kb = kg + (size_t)w.bh * Tlen * dg;
            const __nv_bfloat16* vb = vg + (size_t)w.bh * Tlen * dg;
            const int t0 = w.tb - 12, r_in = lane & 7, cq = lane >> 3;
#pragma unroll 1
            for (int rb = 0; rb < (ST_XROWS + 7) / 8; ++rb) {
                const int r = rb * 8 + r_in, t = t0 + r;
                const bool ok = r < ST_XROWS && t >= 0 && t < Tlen;
                if (r < ST_XROWS) {
#pragma unroll
                    for (int cg = 0; cg < 4; ++cg) {
                        const int c = cg * 4 + cq;
                        const bool real = ok && (c & 7) * 8 < dg;   // channels past the head dimension are zero-filled
                        const __nv_bfloat16* src = (cg < 2 ? kb : vb) + (size_t)(real ? t : 0) * dg + (real ? (c & 7) * 8 : 0);
                        cp_async16(sX + c * ST_COL + r * 16, src, real ? 16u : 0u);
                    }
                }
            }
            cp_async_commit();
            cp_async_wait<0>();
            fence_proxy_async();                               // the tensor core reads these rows through the async proxy
            __syncwarp();
            if (leader) mbar_arrive(bar_x);
        };
        auto load_tap = [&](int n, int h) {                    // n: taps since the start of this CTA's walk (3 per tile)
            if (leader) {
                const uint32_t bar = bar_rf + 8 * (n & 1);
                mbar_expect_tx(bar, IMG_W0_TAP);
                bulk_g2s(sRing + (n & 1) * IMG_W0_TAP, img + (size_t)h * IMG_HEAD + (size_t)(n % 3) * IMG_W0_TAP, IMG_W0_TAP, bar);
            }
        };
        auto load_head = [&](int h) {
            if (leader) {
                mbar_expect_tx(bar_w, IMG_RES);
                bulk_g2s(sW1, img + (size_t)h * IMG_HEAD + IMG_W0, IMG_RES, bar_w);
            }
        };
        // a ring slot is free once the MMAs of the tap it held have completed; every tap is awaited once, in order
        auto wait_tap_done = [&](int n) { swait(bar_re + 8 * (n & 1), (n >> 1) & 1, 20); };
        if (n_my > 0) {
            StackWork w = stack_work(f_begin, n_t, B, H);
            int h_loaded = w.h;
            load_head(w.h);
            load_tap(0, w.h); load_tap(1, w.h);
            load_x(w);
            wait_tap_done(0);
            load_tap(2, w.h);
            for (int it = 0; it < n_my; ++it) {
                const bool more = it + 1 < n_my;
                StackWork wn = w;
                if (more) wn = stack_work(f_begin + it + 1, n_t, B, H);
                if (more) {
                    wait_tap_done(3 * it + 1);
                    load_tap(3 * it + 3, wn.h);
                    wait_tap_done(3 * it + 2);                 // the first layer of tile it is done: the input buffer takes the next tile
                    load_tap(3 * it + 4, wn.h);
                    load_x(wn);
                    wait_tap_done(3 * it + 3);
                    load_tap(3 * it + 5, wn.h);
                } else {
                    wait_tap_done(3 * it + 1);
                    wait_tap_done(3 * it + 2);
                }
                // The resident weights change with the head, once every reader of the old ones is done with the previous
                // tile.  That tile's end is awaited here, one tile late, where it no longer holds up the loads above; the
                // epilogue of a head's first tile waits for the new weights.  While this warp waits for the end of tile
                // it-1, the epilogues can get as far as the end of tile it+1 (whose loads are out), so the barrier is one
                // of four by tile number: with fewer, a late waiter would take a later completion for the one it wants.
                if (it >= 1) {
                    swait(bar_ed4 + 8 * ((it - 1) & 3), ((it - 1) >> 2) & 1, 22);
                    if (w.h != h_loaded) { load_head(w.h); h_loaded = w.h; }
                }
                w = wn;
            }
        }
    } else if (warp == 8) {
        // =================================== MMA issue, first layer ========================================
        // Two warps issue MMAs (an issue costs some 50 cycles, more than the small products of the later layers take):
        // this one the first layer, one tile ahead of the epilogues and into the other of two accumulators; warp 10 the
        // second and third layers.  The whole warp walks the schedule; only the tcgen05 instructions are issued by lane 0.
        const bool leader = lane == 0;
        constexpr uint32_t LBO_X = ST_COL, LBO_W0 = 192 * 16;
        for (int it = 0; it < n_my; ++it) {
            // this accumulator was last used by tile it-2: its epilogue has loaded it.  (Barriers per accumulator: this
            // warp runs up to two tiles ahead of the epilogues, and a barrier must never get two phases ahead of a waiter.)
            if (it >= 2) swait(bar_f0 + 8 * (it & 1), ((it >> 1) - 1) & 1, 6);
            swait(bar_x, it & 1, 1);
            STP(0);
            for (int tau = 0; tau < 3; ++tau) {
                const int n = 3 * it + tau;
                swait(bar_rf + 8 * (n & 1), (n >> 1) & 1, 2);
                tc_fence_after();
                const uint32_t a0 = desc_lo(sX + 2 * tau * 16, LBO_X), b0 = desc_lo(sRing + (n & 1) * IMG_W0_TAP, LBO_W0);
                const uint32_t d = tmem + D0_COL + (it & 1) * 192;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t ad = desc64(a0 + ((2 * kk * ST_COL) >> 4), kDescHiFlat), bd = desc64(b0 + ((2 * kk * 192 * 16) >> 4), kDescHiFlat);
                    if (leader) umma(d, ad, bd, instr_desc(128, 192, false), (tau > 0 || kk > 0) ? 1u : 0u);
                }
                if (leader) {
                    umma_commit(bar_re + 8 * (n & 1));
                    if (tau == 2) umma_commit((it & 1) ? bar_d0b : bar_d0);
                }
                __syncwarp();
            }
            STP(2);
        }
    } else if (warp == 10) {
        // =================================== MMA issue, second and third layers ============================
        const bool leader = lane == 0;
        constexpr uint32_t LBO_X = ST_COL, LBO_W1 = 96 * 16, LBO_W2 = 48 * 16;
        int heads_seen = 0, h_prev = -1;
        for (int it = 0; it < n_my; ++it) {
            const StackWork w = stack_work(f_begin + it, n_t, B, H);
            if (w.h != h_prev) { swait(bar_w, heads_seen & 1, 3); ++heads_seen; h_prev = w.h; }   // this head's small layers are in
            // ---- layer 1: taps x activation pieces (N = 96, 64, 32: the weight pieces each one meets) x 4 K steps ----
            swait(bar_h0, it & 1, 4);
            STP(3);
            tc_fence_after();
#pragma unroll
            for (int tau = 0; tau < 3; ++tau) {
#pragma unroll
                for (int p = 0; p < 3; ++p) {
                    const uint32_t a1 = desc_lo(sH0 + p * 8 * ST_COL + (4 + 2 * tau) * 16, LBO_X);
                    const uint32_t b1 = desc_lo(sW1 + tau * 8 * 96 * 16, LBO_W1);
                    const uint32_t idesc = p == 0 ? instr_desc(128, 96, false) : p == 1 ? instr_desc(128, 64, false) : instr_desc(128, 32, false);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint64_t ad = desc64(a1 + ((2 * kk * ST_COL) >> 4), kDescHiFlat), bd = desc64(b1 + ((2 * kk * 96 * 16) >> 4), kDescHiFlat);
                        if (leader) umma(tmem + D1_COL, ad, bd, idesc, (tau > 0 || p > 0 || kk > 0) ? 1u : 0u);
                    }
                }
            }
            if (leader) umma_commit(bar_d1);
            __syncwarp();
            STP(4);
            // ---- layer 2: N = 48, 32, 16, 2 K steps; its accumulator takes the columns of the second layer's, which the
            // epilogue has read before it publishes h1 ----
            swait(bar_h1, it & 1, 5);
            STP(5);
            tc_fence_after();
#pragma unroll
            for (int tau = 0; tau < 3; ++tau) {
#pragma unroll
                for (int p = 0; p < 3; ++p) {
                    const uint32_t a2 = desc_lo(sH1 + p * 4 * ST_COL + (4 + 2 * tau) * 16, LBO_X);
                    const uint32_t b2 = desc_lo(sW2 + tau * 4 * 48 * 16, LBO_W2);
                    const uint32_t idesc = p == 0 ? instr_desc(128, 48, false) : p == 1 ? instr_desc(128, 32, false) : instr_desc(128, 16, false);
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) {
                        const uint64_t ad = desc64(a2 + ((2 * kk * ST_COL) >> 4), kDescHiFlat), bd = desc64(b2 + ((2 * kk * 48 * 16) >> 4), kDescHiFlat);
                        if (leader) umma(tmem + D2_COL, ad, bd, idesc, (tau > 0 || p > 0 || kk > 0) ? 1u : 0u);
                    }
                }
            }
            if (leader) umma_commit(bar_d2);
            __syncwarp();
            STP(6);
        }
    } else if (warp < 8) {
        // =================================== epilogue warps ================================================
        // warp w owns TMEM lanes 32 (w & 3) .. +31 (row m of the tile) and, where a layer is split, half (w >> 2) of its channels
        const int q = warp & 3, half = warp >> 2;
        const int m = q * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(q * 32)) << 16;
        const uint32_t row_off = (uint32_t)(8 + m) * 16;       // hidden rows sit 8 rows down their columns
        auto f = [](uint32_t u) { return __uint_as_float(u); };
        auto store_chunk = [](uint32_t dst, const uint32_t (&wv)[4]) {
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(wv[0]), "r"(wv[1]), "r"(wv[2]), "r"(wv[3]) : "memory");
        };
        int heads_seen = 0, h_prev = -1;
        for (int it = 0; it < n_my; ++it) {
            const int ff = f_begin + it;
            const StackWork w = stack_work(ff, n_t, B, H);
            const int time = w.tb - 8 + m;
            // every layer's output is zero at negative times (a mask, not a branch: the channels' chains must interleave)
            const uint32_t live_mask = time >= 0 ? 0xffffffffu : 0u;
            if (w.h != h_prev) { swait(bar_w, heads_seen & 1, 10); ++heads_seen; h_prev = w.h; }

            // ---- layer 0 -> h0: 32 of the 64 channels per warp ----
            if (warp == 0) STP(10);
            swait((it & 1) ? bar_d0b : bar_d0, (it >> 1) & 1, 11);
            if (warp == 0) STP(11);
            tc_fence_after();
            {
                uint32_t a[32], b[32], c[32];
                tmem_ld32(tmem + lane_base + D0_COL + (it & 1) * 192 + half * 32, a);
                tmem_ld32(tmem + lane_base + D0_COL + (it & 1) * 192 + 64 + half * 32, b);
                tmem_ld32(tmem + lane_base + D0_COL + (it & 1) * 192 + 128 + half * 32, c);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_f0 + 8 * (it & 1));   // the accumulator may take tile it + 2
                if (warp == 0) STP(20);
                float bias[32];
#pragma unroll
                for (int e = 0; e < 8; ++e) *reinterpret_cast<float4*>(&bias[4 * e]) = *reinterpret_cast<const float4*>(par + half * 32 + 4 * e);
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t hi[4], mid[4], lo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int c0 = ch * 8 + 2 * e;
                        float y0 = (f(a[c0]) + f(b[c0])) + f(c[c0]) + bias[c0];
                        float y1 = (f(a[c0 + 1]) + f(b[c0 + 1])) + f(c[c0 + 1]) + bias[c0 + 1];
                        y0 = __uint_as_float(__float_as_uint(swish(y0)) & live_mask);
                        y1 = __uint_as_float(__float_as_uint(swish(y1)) & live_mask);
                        split3(y0, y1, hi[e], mid[e], lo[e]);
                    }
                    const uint32_t dst = sH0 + (uint32_t)(half * 4 + ch) * ST_COL + row_off;
                    store_chunk(dst, hi); store_chunk(dst + 8 * ST_COL, mid); store_chunk(dst + 16 * ST_COL, lo);
                }
            }
            if (warp == 0) STP(21);
            fence_proxy_async();                               // the tensor core reads these rows through the async proxy
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_h0);
            if (warp == 0) STP(12);

            // ---- layer 1 -> h1: 16 of the 32 channels per warp ----
            swait(bar_d1, it & 1, 12);
            if (warp == 0) STP(13);
            tc_fence_after();
            {
                uint32_t a[16], b[16], c[16];
                tmem_ld16(tmem + lane_base + D1_COL + half * 16, a);
                tmem_ld16(tmem + lane_base + D1_COL + 32 + half * 16, b);
                tmem_ld16(tmem + lane_base + D1_COL + 64 + half * 16, c);
                tmem_wait_ld();
                float bias[16];
#pragma unroll
                for (int e = 0; e < 4; ++e) *reinterpret_cast<float4*>(&bias[4 * e]) = *reinterpret_cast<const float4*>(par + 64 + half * 16 + 4 * e);
#pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    uint32_t hi[4], mid[4], lo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int c0 = ch * 8 + 2 * e;
                        float y0 = (f(a[c0]) + f(b[c0])) + f(c[c0]) + bias[c0];
                        float y1 = (f(a[c0 + 1]) + f(b[c0 + 1])) + f(c[c0 + 1]) + bias[c0 + 1];
                        y0 = __uint_as_float(__float_as_uint(swish(y0)) & live_mask);
                        y1 = __uint_as_float(__float_as_uint(swish(y1)) & live_mask);
                        split3(y0, y1, hi[e], mid[e], lo[e]);
                    }
                    const uint32_t dst = sH1 + (uint32_t)(half * 2 + ch) * ST_COL + row_off;
                    store_chunk(dst, hi); store_chunk(dst + 4 * ST_COL, mid); store_chunk(dst + 8 * ST_COL, lo);
                }
            }
            fence_proxy_async();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_h1);
            if (warp == 0) STP(14);

            // ---- layer 2 and the output map: warps 0-3, one logit per row.  Every warp waits for the third layer: it reads
            // h1 from the columns that the next tile's h0 goes to ----
            swait(bar_d2, it & 1, 13);
            if (half == 0) {
                if (warp == 0) STP(15);
                tc_fence_after();
                uint32_t a[16], b[16], c[16];
                tmem_ld16(tmem + lane_base + D2_COL, a);
                tmem_ld16(tmem + lane_base + D2_COL + 16, b);
                tmem_ld16(tmem + lane_base + D2_COL + 32, c);
                tmem_wait_ld();
                if (warp == 0) STP(17);
                float pv[32];                                  // b2[16] | wout[16]
#pragma unroll
                for (int e = 0; e < 8; ++e) *reinterpret_cast<float4*>(&pv[4 * e]) = *reinterpret_cast<const float4*>(par + 96 + 4 * e);
                float zq[4] = {par[128], 0.f, 0.f, 0.f};
#pragma unroll
                for (int c0 = 0; c0 < 16; ++c0) {
                    float y = (f(a[c0]) + f(b[c0])) + f(c[c0]) + pv[c0];
                    y = __uint_as_float(__float_as_uint(swish(y)) & live_mask);
                    zq[c0 & 3] = fmaf(pv[16 + c0], y, zq[c0 & 3]);
                }
                const float zz = (zq[0] + zq[1]) + (zq[2] + zq[3]);
                if (warp == 0) STP(18);
                const int j = time - ST_HALF;                  // the logit of token j is the output at time j + 6
                if (m >= 8 && time < Tlen) {
                    z[(size_t)w.bh * Tlen + j] = zz;
                    if (r_out) r_out[(size_t)w.bh * Tlen + j] = 1.f / (1.f + expf(-zz));
                }
                // the last tile of a row also marks the six tokens whose right context does not exist yet
                if ((ff + 1) % n_t == 0 && warp == 0 && lane < ST_HALF && Tlen - ST_HALF + lane >= 0) {
                    z[(size_t)w.bh * Tlen + Tlen - ST_HALF + lane] = -INFINITY;
                    if (r_out) r_out[(size_t)w.bh * Tlen + Tlen - ST_HALF + lane] = 0.f;
                }
                if (warp == 0) STP(19);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_ed4 + 8 * (it & 3));
                if (warp == 0) STP(16);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, ST_TMEM);
}

}  // namespace

int stack_tc_status_fetch_and_clear() { return status_fetch_and_clear(g_stack_tc_status); }

// Workspace of the tensor-core stack scorer (the split weight image), 0 where that path does not apply.
size_t scores_stack_tc_workspace(const Params& p)
{
    if (p.dtype != LTE_BF16 || (p.d != ST_D && p.d != 32) || p.T <= 2 * ST_HALF) return 0;
    return (size_t)p.H * IMG_HEAD;
}

// LTE_ERR_UNSUPPORTED where the path does not apply or the workspace is too small (the caller then runs the fp32 kernel).
int launch_scores_stack_tc(const Params& p, const void* k, const void* v, float* z, float* r, void* ws, size_t ws_bytes,
                           cudaStream_t st)
{
    const size_t need = scores_stack_tc_workspace(p);
    if (need == 0 || !ws || ws_bytes < need || ((uintptr_t)ws & 127u) != 0) return LTE_ERR_UNSUPPORTED;
    static PerDeviceOnce attr;
    if (int e = attr.run([] { return cudaFuncSetAttribute(scores_stack_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ST_SMEM); })) return e;
    int n_sm = 0;
    if (int e = device_sm_count(&n_sm)) return e;
    const int BH = p.B * p.H;
    if (launch_pdl(stack_image_kernel, dim3(p.H, 32), dim3(256), 0, st, p.w, p.bias, (uint8_t*)ws, p.H, p.d) != cudaSuccess) return LTE_ERR_CUDA;
    const int n_t = (p.T - ST_HALF + ST_VALID - 1) / ST_VALID;
    const long long n_flat = (long long)BH * n_t;
    if (n_flat > 0x7fffffffLL) return LTE_ERR_UNSUPPORTED;
    const int grid = (int)(n_flat < n_sm ? n_flat : n_sm);
    const int per = (int)((n_flat + grid - 1) / grid);
    const int n_cta = (int)((n_flat + per - 1) / per);
    if (launch_pdl(scores_stack_tc_kernel, dim3(n_cta), dim3(ST_THREADS), ST_SMEM, st, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const uint8_t*)ws, z, r, p.B, p.H,
                   p.T, n_t, (int)n_flat, per, p.d) != cudaSuccess)
        return LTE_ERR_CUDA;
    return cuda_status(cudaGetLastError());
}

}  // namespace lte

#ifdef LTE_PROFILE
extern "C" int lte_stack_status_raw() { return lte::stack_tc_status_fetch_and_clear(); }
extern "C" int lte_stprof_read(long long* out)
{
    return cudaMemcpyFromSymbol(out, lte::g_stprof, sizeof(long long) * 64) == cudaSuccess ? 0 : -1;
}
#endif
