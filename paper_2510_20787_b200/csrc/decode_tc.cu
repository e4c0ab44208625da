// Decode step on the tensor cores (bf16, d = 64, W + R <= 256): Fig. 3's cache, Section 3.1.3's decoding paragraph.
//
// The per-head cache block stores its key and value rows with the 128-byte swizzle, so that once cp.async.bulk has
// copied the block into shared memory it is a valid tcgen05 operand as it stands:
//   logits   S^T[256 keys] = K[256 x 64] q[64]:  two MMAs-groups M = 128 (keys), N = 16 (row 0 of B is q, the rest 0),
//            K = 64; the logit of key j lands in TMEM lane j mod 128, and the thread owning that lane masks it
//            (ring / pool validity after the replacement decision), takes part in the block max / sum and writes
//            p_j = exp(s_j - max) as bf16 into a small B tile;
//   output   O[64] = sum_j p_j V_j:  one MMA chain M = 128 = two stacked halves of 64 channels (A = the value block as
//            MN-major operand: group 0 = rows 0..127, group 1 = rows 128..255), N = 16 (B row 0 = p[0..127],
//            row 1 = p[128..255]), K = 128 keys; channel c is D[c][0] + D[64+c][1].
// Persistent CTAs walk consecutive heads; a control lane issues the bulk copies (next head's keys as soon as this
// head's logits are taken, next values after the PV chain) and every tcgen05.mma; the replacement decision, the
// scorer tap sums and the write-back stay as in the ALU kernel.  Every wait is bounded.
#include "tc_common.cuh"

namespace lte {

__device__ StatusWord g_decode_tc_status = LTE_STATUS_INIT;

namespace {

using namespace tc;
constexpr int NC = 256;                    // compute threads: thread j owns cache row j
constexpr int NTHR = NC + 32;              // + control warp
constexpr int D = 64;
constexpr uint32_t TMEM_COLS = 64;         // S^T: [0,16) keys 0..127, [16,32) keys 128..255;  O halves: [32,48)

__device__ __forceinline__ void dwait(uint32_t bar, uint32_t parity, int code) { mbar_wait_s(bar, parity, code, &g_decode_tc_status); }
__device__ __forceinline__ void csync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

struct Plan { uint32_t off_v, off_tail, tail_bytes, off_q, off_p, off_bar, total; };
__host__ __device__ inline Plan plan_of(const CacheLayout& L) {
    Plan P;
    P.off_v = 32768;                                   // K block [256][64] bf16, then V block
    P.off_q = 65536;                                   // B operand of the logits: [16][64] bf16 (2 KB)
    P.off_p = P.off_q + 2048;                          // B operand of the PV chain: [2][16][64] bf16 (4 KB)
    P.off_tail = P.off_p + 4096;                       // two tail buffers
    P.tail_bytes = (uint32_t)(L.stride - L.off_z);
    P.off_bar = (P.off_tail + 2 * P.tail_bytes + 15) & ~15u;
    P.total = P.off_bar + 128;
    return P;
}

__global__ void __launch_bounds__(NTHR) decode_tc_kernel(unsigned char* __restrict__ cache, CacheLayout L,
                                                         const __nv_bfloat16* __restrict__ q1,
                                                         const __nv_bfloat16* __restrict__ k1,
                                                         const __nv_bfloat16* __restrict__ v1,
                                                         __nv_bfloat16* __restrict__ o1, float* __restrict__ lse1,
                                                         const float* __restrict__ cw, const float* __restrict__ cbias,
                                                         int BH, int per_cta, int H, int W, int R, int sink, int K,
                                                         float zthr, float scale, int G)
{
    extern __shared__ __align__(1024) unsigned char dsm[];
    const Plan P = plan_of(L);
    const uint32_t base = smem_u32(dsm);
    if ((base & 1023u) != 0) { if (threadIdx.x == 0) atomicExch(&g_decode_tc_status.code, 9); return; }
    const uint32_t sK = base, sV = base + P.off_v, sT = base + P.off_tail, sQ = base + P.off_q, sP = base + P.off_p;
    const uint32_t bar_k = base + P.off_bar, bar_v = bar_k + 8, bar_t0 = bar_k + 16;     // bar_t0, bar_t0 + 8
    const uint32_t bar_q = bar_k + 32, bar_s = bar_k + 40, bar_p = bar_k + 48, bar_o = bar_k + 56, tmem_slot = bar_k + 64;
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(dsm + P.off_bar + 64);
    __shared__ float s_part[8], s_sum[8], s_tap[kMaxTaps], s_o[128];

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int rows = W + R, half = K / 2;
    const int bh_begin = blockIdx.x * per_cta;
    const int bh_end = min(bh_begin + per_cta, BH);
    if (bh_begin >= bh_end) return;

    if (tid == 0) {
        mbar_init(bar_k, 1); mbar_init(bar_v, 1); mbar_init(bar_t0, 1); mbar_init(bar_t0 + 8, 1);
        mbar_init(bar_q, 8); mbar_init(bar_s, 1); mbar_init(bar_p, NC); mbar_init(bar_o, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // the two small B tiles start as zeros (only row 0 of the q tile and rows 0, 1 of the p tile are ever written)
    for (int e = tid; e < (2048 + 4096) / 16; e += NTHR)
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(sQ + e * 16), "r"(0u) : "memory");
    if (wid == 8) tmem_alloc(tmem_slot, TMEM_COLS);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;
    pdl_launch_dependents();
    pdl_wait();                                                // the previous step (or whatever wrote the cache and the inputs) has completed

    if (wid == 8) {
        // ======================================== control lane ==================================================
        if (lane == 0) {
            constexpr uint32_t IDESC_S = instr_desc(128, 16, false);
            constexpr uint32_t IDESC_O = instr_desc(128, 16, false, true);        // A (values) MN-major, B (p) K-major
            const uint32_t k_lo = desc_lo(sK, 16), q_lo = desc_lo(sQ, 16), vmn_lo = desc_lo(sV, 16384), p_lo = desc_lo(sP, 16);
            const unsigned char* g0 = cache + L.header + (size_t)bh_begin * L.stride;
            bulk_load(sT, g0 + L.off_z, P.tail_bytes, bar_t0);
            bulk_load(sK, g0 + L.off_k, 32768, bar_k);
            bulk_load(sV, g0 + L.off_v, 32768, bar_v);
            for (int bh = bh_begin, it = 0; bh < bh_end; ++bh, ++it) {
                const unsigned char* gnext = cache + L.header + (size_t)(bh + 1) * L.stride;
                dwait(bar_k, it & 1, 1);
                dwait(bar_q, it & 1, 2);                       // q of this head is in the B tile
                tc_fence_after();
#pragma unroll
                for (int g = 0; g < 2; ++g)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma(tmem + g * 16, desc64(k_lo + g * 1024 + kk * 2, kDescHi), desc64(q_lo + kk * 2, kDescHi), IDESC_S, kk > 0);
                umma_commit(bar_s);
                dwait(bar_p, it & 1, 3);                       // p is in its B tile; the key block is no longer read by anyone
                if (bh + 1 < bh_end) bulk_load(sK, gnext + L.off_k, 32768, bar_k);
                dwait(bar_v, it & 1, 4);
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)                 // 128 keys per half, 16 per instruction
                    umma(tmem + 32, desc64(vmn_lo + kk * 128, kDescHi), desc64(p_lo + (kk >> 2) * 128 + (kk & 3) * 2, kDescHi),
                         IDESC_O, kk > 0);
                umma_commit(bar_o);
                if (bh + 1 < bh_end) {
                    dwait(bar_o, it & 1, 5);                   // the value block has been consumed
                    bulk_load(sV, gnext + L.off_v, 32768, bar_v);
                    bulk_load(sT + ((it & 1) ^ 1) * P.tail_bytes, gnext + L.off_z, P.tail_bytes, bar_t0 + 8 * ((it & 1) ^ 1));
                }
            }
        }
    } else {
        // ======================================== compute threads ===============================================
        constexpr int CPL = D / 32;            // channels per lane in the warp-per-row pieces
        const uint32_t lane_base = ((uint32_t)((wid & 3) * 32)) << 16;
        float k1f[CPL], v1f[CPL], q1f[CPL], wk[2][CPL], wv[2][CPL], bias = 0.f, v1_mine = 0.f;
        uint4 kv_new = make_uint4(0, 0, 0, 0), q_chunk = make_uint4(0, 0, 0, 0);
        auto fetch_inputs = [&](int bh) {
            const int h = bh % H;
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                k1f[c] = __bfloat162float(k1[(size_t)bh * D + lane + 32 * c]);
                v1f[c] = __bfloat162float(v1[(size_t)bh * D + lane + 32 * c]);
                q1f[c] = __bfloat162float(q1[(size_t)bh * G * D + lane + 32 * c]);
            }
#pragma unroll
            for (int u2 = 0; u2 < 2; ++u2) {
                const int t = wid + u2 * 8;
#pragma unroll
                for (int c = 0; c < CPL; ++c) {
                    wk[u2][c] = t < K ? cw[((size_t)h * K + t) * 2 * D + lane + 32 * c] : 0.f;
                    wv[u2][c] = t < K ? cw[((size_t)h * K + t) * 2 * D + D + lane + 32 * c] : 0.f;
                }
            }
            bias = cbias ? cbias[h] : 0.f;
            if (tid < D) v1_mine = __bfloat162float(v1[(size_t)bh * D + tid]);
            if (tid < 8) q_chunk = *reinterpret_cast<const uint4*>(q1 + (size_t)bh * G * D + tid * 8);
            if (tid >= 64 && tid < 80) {
                const int t2 = tid - 64;
                kv_new = *reinterpret_cast<const uint4*>((t2 < 8 ? k1 : v1) + (size_t)bh * D + (t2 & 7) * 8);
            }
        };
        fetch_inputs(bh_begin);

        for (int bh = bh_begin, it = 0; bh < bh_end; ++bh, ++it) {
            const int tb = it & 1;
            unsigned char* gblk = cache + L.header + (size_t)bh * L.stride;
            // q -> row 0 of the logits' B tile (row 0 of a swizzled tile is stored in order)
            if (tid < 8) {
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sQ + tid * 16), "r"(q_chunk.x), "r"(q_chunk.y),
                             "r"(q_chunk.z), "r"(q_chunk.w) : "memory");
                fence_proxy_async();
                mbar_arrive(bar_q);
            }
            dwait(bar_t0 + 8 * tb, (it >> 1) & 1, 6);
            const unsigned char* tail = dsm + P.off_tail + (size_t)tb * P.tail_bytes;
            const float* zc = reinterpret_cast<const float*>(tail);
            const int32_t* pidx = reinterpret_cast<const int32_t*>(tail + (L.off_pidx - L.off_z));
            const int32_t* meta = reinterpret_cast<const int32_t*>(tail + (L.off_meta - L.off_z));
            const int n = meta[0], cnt_old = meta[1];
            const int slot = n % W;

            // ---- pool decision, taken redundantly by every warp so that the row masks are known early -----------
            int dst = -1, cnt_new = cnt_old;
            {
                const int p = n - W;
                if (p >= 0 && R > 0) {
                    const float zp = zc[slot];
                    const bool is_sink = p < sink;
                    if (is_sink || zp > zthr) {
                        if (cnt_old < R) { dst = cnt_old; cnt_new = cnt_old + 1; }
                        else if (!is_sink) {
                            // worst entry: lowest logit, the youngest among equals, never a sink entry
                            float wz = INFINITY; int wpos = -1, wslot = -1;
                            for (int m = lane; m < cnt_old; m += 32) {
                                const int pos = pidx[m];
                                const float zm = zc[W + m];
                                if (pos >= sink && (zm < wz || (zm == wz && pos > wpos))) { wz = zm; wpos = pos; wslot = m; }
                            }
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) {
                                const float oz = __shfl_xor_sync(0xffffffffu, wz, o);
                                const int op = __shfl_xor_sync(0xffffffffu, wpos, o);
                                const int os = __shfl_xor_sync(0xffffffffu, wslot, o);
                                if (os >= 0 && (wslot < 0 || oz < wz || (oz == wz && op > wpos))) { wz = oz; wpos = op; wslot = os; }
                            }
                            if (wslot >= 0 && zp > wz) dst = wslot;
                        }
                    }
                }
            }
            // ---- direct reads of the key / value blocks: scorer taps and the popped row ----------------------
            dwait(bar_k, it & 1, 7);
            dwait(bar_v, it & 1, 8);
            const int jsc = K > 0 ? n - half : -1;   // K = 0: the scorer runs outside (lte_cache_score)
            if (jsc >= 0) {
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int t = wid + u * 8;
                    if (t >= K) continue;
                    const int pos = jsc + t - half;
                    float a = 0.f;
                    if (pos == n) {
#pragma unroll
                        for (int c = 0; c < CPL; ++c) a += wk[u][c] * k1f[c] + wv[u][c] * v1f[c];
                    } else if (pos >= 0) {
                        const int rr = pos % W;
#pragma unroll
                        for (int c = 0; c < CPL; ++c) {
                            const int ch = lane + 32 * c;          // channel -> swizzled element index within the row
                            const int el = (((ch >> 3) ^ (rr & 7)) << 3) | (ch & 7);
                            const float kx = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(dsm)[rr * D + el]);
                            const float vx = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(dsm + P.off_v)[rr * D + el]);
                            a += wk[u][c] * kx + wv[u][c] * vx;
                        }
                    }
                    a = warp_sum(a);
                    if (lane == 0) s_tap[t] = a;
                }
            }
            // the popped row doubles as the new pool entry: logical chunk c of row `slot`, kept in a register
            uint4 mv = make_uint4(0, 0, 0, 0);
            if (tid < 16)
                mv = reinterpret_cast<const uint4*>(dsm + (tid < 8 ? 0 : P.off_v))[(size_t)slot * 8 + ((tid & 7) ^ (slot & 7))];
            float s_new = 0.f;                                 // logit of the incoming token (every warp computes it)
#pragma unroll
            for (int c = 0; c < CPL; ++c) s_new = fmaf(q1f[c], k1f[c], s_new);
            s_new = warp_sum(s_new) * scale;

            // ---- logits from TMEM, masks, softmax --------------------------------------------------------------
            dwait(bar_s, it & 1, 9);
            tc_fence_after();
            uint32_t sraw;
            tmem_ld1(tmem + lane_base + (tid >> 7) * 16, sraw);
            tmem_wait_ld();
            const int row = tid;
            bool ok;
            if (row >= rows) ok = false;
            else if (row < W) ok = (n >= W) ? (row != slot || dst >= 0) : (row < n);
            else ok = (row - W) < cnt_old && (row - W) != dst;
            const float sl = ok ? __uint_as_float(sraw) * scale : -INFINITY;
            float mx = warp_max(fmaxf(sl, s_new));
            if (lane == 0) s_part[wid] = mx;
            csync();
            mx = s_part[0];
#pragma unroll
            for (int w2 = 1; w2 < 8; ++w2) mx = fmaxf(mx, s_part[w2]);
            // p rounded to bf16: the same rounded values enter the product and the normalisation
            const __nv_bfloat16 pb = __float2bfloat16_rn(__expf(sl - mx));
            {
                const int rr = row >> 7, col = row & 127, c64 = col & 63;
                const uint32_t off = (col >> 6) * 2048 + rr * 128 + ((((c64 >> 3) ^ (rr & 7))) << 4) + (c64 & 7) * 2;
                asm volatile("st.shared.b16 [%0], %1;" ::"r"(sP + off), "h"(*reinterpret_cast<const unsigned short*>(&pb)) : "memory");
            }
            float lsum = warp_sum(__bfloat162float(pb));
            if (lane == 0) s_sum[wid] = lsum;
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar_p);

            // ---- output ----------------------------------------------------------------------------------------
            dwait(bar_o, it & 1, 10);
            tc_fence_after();
            if (tid < 128) {
                uint32_t oraw;
                tmem_ld1(tmem + lane_base + 32 + (tid >> 6), oraw);   // lanes 0..63: column 0, lanes 64..127: column 1
                tmem_wait_ld();
                s_o[tid] = __uint_as_float(oraw);
            }
            tc_fence_before();
            csync();
            const float p_new = __expf(s_new - mx);
            float sum = p_new;
#pragma unroll
            for (int w2 = 0; w2 < 8; ++w2) sum += s_sum[w2];
            if (tid < D) {
                const float o = s_o[tid] + s_o[64 + tid] + p_new * v1_mine;
                o1[(size_t)bh * G * D + tid] = __float2bfloat16_rn(o / sum);
            }
            if (tid == 0) lse1[(size_t)bh * G] = mx + logf(sum);

            // ---- write-back: only what changed goes to HBM (rows are stored swizzled) ----------------------------
            uint4* Kw = reinterpret_cast<uint4*>(gblk + L.off_k);
            uint4* Vw = reinterpret_cast<uint4*>(gblk + L.off_v);
            float* zw = reinterpret_cast<float*>(gblk + L.off_z);
            int32_t* pw = reinterpret_cast<int32_t*>(gblk + L.off_pidx);
            int32_t* mw = reinterpret_cast<int32_t*>(gblk + L.off_meta);
            if (dst >= 0 && tid < 16) {
                const int rr = W + dst;
                (tid < 8 ? Kw : Vw)[(size_t)rr * 8 + ((tid & 7) ^ (rr & 7))] = mv;
            }
            if (tid >= 64 && tid < 80) {
                const int t2 = tid - 64;
                (t2 < 8 ? Kw : Vw)[(size_t)slot * 8 + ((t2 & 7) ^ (slot & 7))] = kv_new;
            }
            if (tid == 128) {
                if (dst >= 0) { zw[W + dst] = zc[slot]; pw[dst] = n - W; }
                float znew = -INFINITY;
                if (jsc >= 0) {
                    znew = bias;
                    for (int t = 0; t < K; ++t) znew += s_tap[t];
                }
                zw[slot] = -INFINITY;
                if (jsc >= 0) zw[jsc % W] = znew;
                mw[0] = n + 1;
                mw[1] = cnt_new;
            }
            csync();                                           // shared scratch is reused by the next head
            if (bh + 1 < bh_end) fetch_inputs(bh + 1);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (wid == 8) tmem_dealloc(tmem, TMEM_COLS);
}

}  // namespace

int launch_decode_tc(const Params& p, void* cache, const void* q1, const void* k1, const void* v1, void* o1, float* lse1,
                     cudaStream_t st)
{
    const CacheLayout L = cache_layout(p.d, p.W, p.R, p.dtype);
    if (!L.swz || p.K > 16) return LTE_ERR_UNSUPPORTED;
    const Plan P = plan_of(L);
    static PerDeviceOnce attr;
    if (int e = attr.run([] { return cudaFuncSetAttribute(decode_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024); })) return e;
    int n_sm = 0;
    if (int e = device_sm_count(&n_sm)) return e;
    if (P.total > 80 * 1024) return LTE_ERR_UNSUPPORTED;
    const int BH = p.B * p.H;
    const int slots = 3 * n_sm;                                // three CTAs per SM
    const int per_cta = (BH + slots - 1) / slots;
    const int n_cta = (BH + per_cta - 1) / per_cta;
    return cuda_status(launch_pdl(decode_tc_kernel, dim3(n_cta), dim3(NTHR), P.total, st, (unsigned char*)cache, L, (const __nv_bfloat16*)q1,
                                                   (const __nv_bfloat16*)k1, (const __nv_bfloat16*)v1, (__nv_bfloat16*)o1, lse1,
                                                   p.w, p.bias, BH, per_cta, p.H, p.W, p.R, p.sink, p.K, p.zthr, p.scale, p.G));
}

int decode_tc_status_fetch_and_clear() { return status_fetch_and_clear(g_decode_tc_status); }

}  // namespace lte
