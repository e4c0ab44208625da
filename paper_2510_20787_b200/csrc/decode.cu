// Decode step over the constant-size per-head cache (Fig. 3; Section 3.1.3, decoding paragraph),
// plus the kernel that builds the cache after a prompt.
//
// One block per (b,h).  All key/value traffic is issued up front as 128-bit coalesced loads of the
// OLD cache rows (their addresses depend on nothing but the layout), while one warp reads the head's
// metadata and decides what happens to the token leaving the window; the decision only turns into
// row masks before the softmax.  The old ring row being popped doubles as the new pool entry when it
// is retained, and the incoming token's row comes from the call's inputs, so no row is read twice.
// Scores: partial dot per lane, shuffle-reduce over the lanes sharing a row; softmax over at most
// W+R+1 logits in shared memory; PV partial sums reduced by shuffles then across warps.  The cache
// write-back (pool slot, ring slot, new logit, counters) is off the critical path at the end.
#include <cooperative_groups.h>

#include "common.cuh"

namespace lte {
namespace cg = cooperative_groups;
namespace {

constexpr int DT = 256;           // threads per block
constexpr int MAX_ROWS = 4096;    // W + R limit of the decode kernel (logits live in shared memory)
constexpr int NCH = 8;            // 16-byte chunks a thread keeps in flight per tensor

template <typename T> struct V16 { static constexpr int N = 16 / sizeof(T); };

template <typename T> __device__ __forceinline__ void unpack(const uint4& u, float* f);
template <> __device__ __forceinline__ void unpack<__nv_bfloat16>(const uint4& u, float* f) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
}
template <> __device__ __forceinline__ void unpack<float>(const uint4& u, float* f) {
    f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y); f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
}

template <typename T, int D>
__global__ void __launch_bounds__(DT) decode_kernel(unsigned char* __restrict__ cache, CacheLayout L,
                                                    const T* __restrict__ q1, const T* __restrict__ k1,
                                                    const T* __restrict__ v1, T* __restrict__ o1,
                                                    float* __restrict__ lse1, const float* __restrict__ cw,
                                                    const float* __restrict__ cbias, int H, int W, int R, int sink,
                                                    int K, float zthr, float scale, int G)
{
    constexpr int EPV = V16<T>::N;            // elements per 16-byte vector
    constexpr int LPR = D / EPV;              // lanes per row
    constexpr int RPP = DT / LPR;             // rows per pass of the whole block
    __shared__ float s_log[MAX_ROWS + 1];
    __shared__ float s_red[DT / 32][D];
    __shared__ float s_part[DT / 32];
    __shared__ float s_tap[kMaxTaps];
    __shared__ int s_dec[4];                  // n, cnt_old, dst (-1 none), cnt_new
    __shared__ float s_zp;

    const int bh = blockIdx.x, h = bh % H;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    unsigned char* blk = cache + L.header + (size_t)bh * L.stride;
    const uint4* Kc = reinterpret_cast<const uint4*>(blk + L.off_k);
    const uint4* Vc = reinterpret_cast<const uint4*>(blk + L.off_v);
    float* zc = reinterpret_cast<float*>(blk + L.off_z);
    int32_t* pidx = reinterpret_cast<int32_t*>(blk + L.off_pidx);
    int32_t* meta = reinterpret_cast<int32_t*>(blk + L.off_meta);
    const int rows = W + R;
    const int seg = tid % LPR, rsub = tid / LPR;
    const int half = K / 2;

    // query segment of this thread (pre-scaled)
    float qf[EPV];
    {
        uint4 u = *reinterpret_cast<const uint4*>(q1 + (size_t)bh * G * D + seg * EPV);
        unpack<T>(u, qf);
#pragma unroll
        for (int e = 0; e < EPV; ++e) qf[e] *= scale;
    }

    // ---- issue the first group of K loads, then let warp 0 take the pool decision ---------------
    uint4 kreg[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        const int row = c * RPP + rsub;
        kreg[c] = row < rows ? Kc[(size_t)row * LPR + seg] : make_uint4(0, 0, 0, 0);
    }

    if (wid == 0) {
        const int n = meta[0], cnt = meta[1];
        const int p = n - W;
        int dst = -1, cnt_new = cnt;
        float zp = -INFINITY;
        if (p >= 0 && R > 0) {
            zp = zc[n % W];
            const bool is_sink = p < sink;
            if (is_sink || zp > zthr) {
                if (cnt < R) { dst = cnt; cnt_new = cnt + 1; }
                else if (!is_sink) {
                    // worst entry: lowest logit, the youngest among equals, never a sink entry
                    float wz = INFINITY; int wpos = -1, wslot = -1;
                    for (int m = lane; m < cnt; m += 32) {
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
        if (lane == 0) { s_dec[0] = n; s_dec[1] = cnt; s_dec[2] = dst; s_dec[3] = cnt_new; s_zp = zp; }
    }

    // ---- phase A: logits of every old row -----------------------------------------------------
    for (int r0 = 0; r0 < rows; r0 += NCH * RPP) {
        if (r0 > 0) {
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                const int row = r0 + c * RPP + rsub;
                kreg[c] = row < rows ? Kc[(size_t)row * LPR + seg] : make_uint4(0, 0, 0, 0);
            }
        }
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            const int row = r0 + c * RPP + rsub;
            float kf[EPV];
            unpack<T>(kreg[c], kf);
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < EPV; ++e) s = fmaf(qf[e], kf[e], s);
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (seg == 0 && row < rows) s_log[row] = s;
        }
    }
    // prefetch the first group of V rows while the softmax is computed
    uint4 vreg[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        const int row = c * RPP + rsub;
        vreg[c] = row < rows ? Vc[(size_t)row * LPR + seg] : make_uint4(0, 0, 0, 0);
    }
    // logit of the incoming token (row index `rows`)
    if (wid == 1) {
        float s = 0.f;
        for (int c = lane; c < D; c += 32) s = fmaf(to_f(q1[(size_t)bh * G * D + c]) * scale, to_f(k1[(size_t)bh * D + c]), s);
        s = warp_sum(s);
        if (lane == 0) s_log[rows] = s;
    }
    __syncthreads();

    const int n = s_dec[0], cnt_old = s_dec[1], dst = s_dec[2], cnt_new = s_dec[3];
    const int slot = n % W;

    // ---- scorer for token j = n - half, from the old ring rows and the incoming row -------------
    const int jsc = K > 0 ? n - half : -1;   // K = 0: the scorer runs outside (lte_cache_score), nothing is scored here
    if (jsc >= 0) {
        for (int t = wid; t < K; t += DT / 32) {
            const int pos = jsc + t - half;
            float a = 0.f;
            if (pos >= 0) {
                const float* wt = cw + ((size_t)h * K + t) * 2 * D;
                if (pos == n) {
                    for (int c = lane; c < D; c += 32)
                        a += wt[c] * to_f(k1[(size_t)bh * D + c]) + wt[D + c] * to_f(v1[(size_t)bh * D + c]);
                } else {
                    const T* kr = reinterpret_cast<const T*>(blk + L.off_k) + (size_t)(pos % W) * D;
                    const T* vr = reinterpret_cast<const T*>(blk + L.off_v) + (size_t)(pos % W) * D;
                    for (int c = lane; c < D; c += 32) a += wt[c] * to_f(kr[c]) + wt[D + c] * to_f(vr[c]);
                }
            }
            a = warp_sum(a);
            if (lane == 0) s_tap[t] = a;
        }
    }

    // ---- masks + softmax over rows+1 logits ---------------------------------------------------
    // old ring row r: token at slot r.  Valid window rows: tokens n-W+1 .. n-1.  The popped row (slot)
    // stays in the sum iff it was accepted into the pool.  Old pool row m: valid iff m < cnt_old and m != dst.
    float mx = -INFINITY;
    for (int r = tid; r <= rows; r += DT) {
        bool ok;
        if (r == rows) ok = true;
        else if (r < W) ok = (n >= W) ? (r != slot || dst >= 0) : (r < n);
        else ok = (r - W) < cnt_old && (r - W) != dst;
        const float s = ok ? s_log[r] : -INFINITY;
        s_log[r] = s;
        mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    if (lane == 0) s_part[wid] = mx;
    __syncthreads();
    mx = s_part[0];
#pragma unroll
    for (int w2 = 1; w2 < DT / 32; ++w2) mx = fmaxf(mx, s_part[w2]);
    __syncthreads();
    float sum = 0.f;
    for (int r = tid; r <= rows; r += DT) {
        const float pr = __expf(s_log[r] - mx);     // exp(-inf) = 0 for masked rows
        s_log[r] = pr;
        sum += pr;
    }
    sum = warp_sum(sum);
    if (lane == 0) s_part[wid] = sum;
    __syncthreads();
    sum = 0.f;
#pragma unroll
    for (int w2 = 0; w2 < DT / 32; ++w2) sum += s_part[w2];
    const float inv = 1.f / sum;

    // ---- phase C: PV --------------------------------------------------------------------------
    float acc[EPV];
#pragma unroll
    for (int e = 0; e < EPV; ++e) acc[e] = 0.f;
    for (int r0 = 0; r0 < rows; r0 += NCH * RPP) {
        if (r0 > 0) {
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                const int row = r0 + c * RPP + rsub;
                vreg[c] = row < rows ? Vc[(size_t)row * LPR + seg] : make_uint4(0, 0, 0, 0);
            }
        }
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            const int row = r0 + c * RPP + rsub;
            const float pr = row < rows ? s_log[row] : 0.f;
            if (pr != 0.f) {
                float vf[EPV];
                unpack<T>(vreg[c], vf);
#pragma unroll
                for (int e = 0; e < EPV; ++e) acc[e] = fmaf(pr, vf[e], acc[e]);
            }
        }
    }
    // rows of the same channel segment sit LPR lanes apart
#pragma unroll
    for (int o = 16; o >= LPR; o >>= 1) {
#pragma unroll
        for (int e = 0; e < EPV; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
    }
    if (lane < LPR) {
#pragma unroll
        for (int e = 0; e < EPV; ++e) s_red[wid][lane * EPV + e] = acc[e];
    }
    // rows needed by the write-back are read before anything is overwritten
    uint4 mv = make_uint4(0, 0, 0, 0);
    if (dst >= 0 && tid < 2 * LPR) mv = (tid < LPR ? Kc : Vc)[(size_t)slot * LPR + (tid % LPR)];
    __syncthreads();

    if (tid < D) {
        float o = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < DT / 32; ++w2) o += s_red[w2][tid];
        o = fmaf(s_log[rows], to_f(v1[(size_t)bh * D + tid]), o);
        o1[(size_t)bh * G * D + tid] = from_f<T>(o * inv);
    }
    if (tid == 0) lse1[(size_t)bh * G] = mx + logf(sum);

    // ---- write-back ---------------------------------------------------------------------------
    uint4* Kw = reinterpret_cast<uint4*>(blk + L.off_k);
    uint4* Vw = reinterpret_cast<uint4*>(blk + L.off_v);
    if (dst >= 0 && tid < 2 * LPR) (tid < LPR ? Kw : Vw)[(size_t)(W + dst) * LPR + (tid % LPR)] = mv;
    if (tid >= 64 && tid < 64 + 2 * LPR) {
        const int t2 = tid - 64;
        const T* src = (t2 < LPR ? k1 : v1) + (size_t)bh * D + (t2 % LPR) * EPV;
        (t2 < LPR ? Kw : Vw)[(size_t)slot * LPR + (t2 % LPR)] = *reinterpret_cast<const uint4*>(src);
    }
    if (tid == 0) {
        if (dst >= 0) { zc[W + dst] = s_zp; pidx[dst] = n - W; }
        float znew = -INFINITY;
        if (jsc >= 0) {
            znew = cbias ? cbias[h] : 0.f;
            for (int t = 0; t < K; ++t) znew += s_tap[t];
        }
        zc[slot] = -INFINITY;                       // the incoming token is not scored yet ...
        if (jsc >= 0) zc[jsc % W] = znew;           // ... unless half == 0 (then jsc == n)
        meta[0] = n + 1;
        meta[1] = cnt_new;
    }
}

// ---- fast path: persistent blocks that stream whole per-head cache blocks through shared memory ------------
// The block of one (b,h) is contiguous in HBM, so three cp.async.bulk copies (TMA, 1-D; mbarrier transaction
// counts) bring its keys, its values and its small tail (logits, pool positions, counters) on chip.  Each CTA
// walks a contiguous range of heads and keeps the copy engine busy: as soon as the logits of head i are done its
// key buffer is refilled with head i+1's keys, and after the PV pass the value buffer is refilled likewise, so
// the loads of the next head run under the softmax / PV / write-back of the current one.  Everything is computed
// out of shared memory; only the rows that change go back to HBM.  Used when a block fits (it does at W+R = 256).
__device__ StatusWord g_decode_status = LTE_STATUS_INIT;   // report only: no wait polls it
#ifdef LTE_PROFILE
__device__ long long g_dprof[64];
#define DPROF(slot) do { if (blockIdx.x == 7 && threadIdx.x == 96 && it == 2) g_dprof[slot] = clock64(); } while (0)
#else
#define DPROF(slot) do { } while (0)
#endif

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Bounded wait; false if it ran out (the caller records it and leaves).
__device__ __forceinline__ bool bar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < (1u << 22); ++it) {
        uint32_t r;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(r) : "r"(bar), "r"(parity) : "memory");
        if (r) return true;
    }
    return false;
}

struct BulkSmem {
    uint32_t kv_bytes, tail_bytes, off_v, off_tail, off_log, off_bar, total;
};
__host__ __device__ inline BulkSmem bulk_smem_plan(const CacheLayout& L, int W, int R) {
    BulkSmem b;
    b.kv_bytes = (uint32_t)L.off_v;                      // bytes of the K rows (= bytes of the V rows)
    b.tail_bytes = (uint32_t)(L.stride - L.off_z);       // logits, pool positions, counters, padding
    b.off_v = b.kv_bytes;
    b.off_tail = 2 * b.kv_bytes;                         // two tail buffers
    b.off_log = b.off_tail + 2 * b.tail_bytes;
    b.off_bar = b.off_log + (uint32_t)(((size_t)W + R + 1) * 4 + 15) / 16 * 16;
    b.total = b.off_bar + 64;
    return b;
}

template <typename T, int D>
__global__ void __launch_bounds__(DT) decode_bulk_kernel(unsigned char* __restrict__ cache, CacheLayout L,
                                                         const T* __restrict__ q1, const T* __restrict__ k1,
                                                         const T* __restrict__ v1, T* __restrict__ o1,
                                                         float* __restrict__ lse1, const float* __restrict__ cw,
                                                         const float* __restrict__ cbias, int BH, int per_cta, int H,
                                                         int W, int R, int sink, int K, float zthr, float scale, int G)
{
    constexpr int EPV = V16<T>::N;
    constexpr int LPR = D / EPV;
    constexpr int RPP = DT / LPR;
    constexpr int CPL = D / 32;                // channels per lane in the warp-per-row pieces
    extern __shared__ __align__(128) unsigned char dsm[];
    const BulkSmem P = bulk_smem_plan(L, W, R);
    const int rows = W + R;
    float* s_log = reinterpret_cast<float*>(dsm + P.off_log);
    const uint32_t bar_k = smem_addr(dsm + P.off_bar), bar_v = bar_k + 8, bar_t0 = bar_k + 16;   // bar_t0, bar_t0 + 8
    __shared__ float s_red[DT / 32][D];
    __shared__ float s_part[DT / 32];
    __shared__ float s_tap[kMaxTaps];
    __shared__ float s_sum[DT / 32];
    __shared__ int s_flag;

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int seg = tid % LPR, rsub = tid / LPR;
    const int half = K / 2;
    const int bh_begin = blockIdx.x * per_cta;
    const int bh_end = min(bh_begin + per_cta, BH);
    if (bh_begin >= bh_end) return;
    const uint32_t sK = smem_addr(dsm), sV = sK + P.off_v, sT = sK + P.off_tail;

    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_k));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_v));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_t0));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_t0 + 8));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const unsigned char* g0 = cache + L.header + (size_t)bh_begin * L.stride;
        bulk_load(sT, g0 + L.off_z, P.tail_bytes, bar_t0);
        bulk_load(sK, g0 + L.off_k, P.kv_bytes, bar_k);
        bulk_load(sV, g0 + L.off_v, P.kv_bytes, bar_v);
    }
    __syncthreads();                                            // barriers initialised before anyone polls them

    // The step's own inputs of a head (query, new key/value, scorer weights) are fetched one head ahead, so
    // their latency hides under the previous head's tail.
    float qf[EPV], k1f[CPL], v1f[CPL], q1f[CPL], wk[2][CPL], wv[2][CPL], bias = 0.f, v1_mine = 0.f;
    uint4 kv_new = make_uint4(0, 0, 0, 0);
    auto fetch_inputs = [&](int bh) {
        const int h = bh % H;
        uint4 u = *reinterpret_cast<const uint4*>(q1 + (size_t)bh * G * D + seg * EPV);
        unpack<T>(u, qf);
#pragma unroll
        for (int c = 0; c < CPL; ++c) {
            k1f[c] = to_f(k1[(size_t)bh * D + lane + 32 * c]);
            v1f[c] = to_f(v1[(size_t)bh * D + lane + 32 * c]);
            q1f[c] = to_f(q1[(size_t)bh * G * D + lane + 32 * c]);
        }
#pragma unroll
        for (int u2 = 0; u2 < 2; ++u2) {
            const int t = wid + u2 * (DT / 32);
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                wk[u2][c] = t < K ? cw[((size_t)h * K + t) * 2 * D + lane + 32 * c] : 0.f;
                wv[u2][c] = t < K ? cw[((size_t)h * K + t) * 2 * D + D + lane + 32 * c] : 0.f;
            }
        }
        bias = cbias ? cbias[h] : 0.f;
        if (tid < D) v1_mine = to_f(v1[(size_t)bh * D + tid]);
        if (tid >= 64 && tid < 64 + 2 * LPR) {
            const int t2 = tid - 64;
            kv_new = *reinterpret_cast<const uint4*>((t2 < LPR ? k1 : v1) + (size_t)bh * D + (t2 % LPR) * EPV);
        }
    };
    fetch_inputs(bh_begin);

    for (int bh = bh_begin, it = 0; bh < bh_end; ++bh, ++it) {
        DPROF(0);
        const int tb = it & 1;
        unsigned char* gblk = cache + L.header + (size_t)bh * L.stride;
        // one thread polls the copy barriers; the block barrier then releases everybody
        if (tid == 0) {
            const bool ok = bar_wait(bar_t0 + 8 * tb, (it >> 1) & 1) && bar_wait(bar_k, it & 1) && bar_wait(bar_v, it & 1);
            s_flag = ok ? 0 : 1;
        }
        __syncthreads();
        if (s_flag) {                                           // bounded wait ran out: give up, outputs undefined
            if (tid == 0) atomicExch(&g_decode_status.code, 1);
            return;
        }
        DPROF(1);
        const uint4* Kc = reinterpret_cast<const uint4*>(dsm);
        const uint4* Vc = reinterpret_cast<const uint4*>(dsm + P.off_v);
        const unsigned char* tail = dsm + P.off_tail + (size_t)tb * P.tail_bytes;
        const float* zc = reinterpret_cast<const float*>(tail);
        const int32_t* pidx = reinterpret_cast<const int32_t*>(tail + (L.off_pidx - L.off_z));
        const int32_t* meta = reinterpret_cast<const int32_t*>(tail + (L.off_meta - L.off_z));
        const int n = meta[0], cnt_old = meta[1];
        const int slot = n % W;

        // ---- pool decision, taken redundantly by every warp so that the row masks are known before the logits --
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
        DPROF(2);
        // ---- scorer taps (warp w owns taps w and w + 8) and the logit of the incoming token (last warp) ----
        const int jsc = K > 0 ? n - half : -1;   // K = 0: the scorer runs outside (lte_cache_score)
        if (jsc >= 0) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int t = wid + u * (DT / 32);
                if (t >= K) continue;
                const int pos = jsc + t - half;
                float a = 0.f;
                if (pos == n) {
#pragma unroll
                    for (int c = 0; c < CPL; ++c) a += wk[u][c] * k1f[c] + wv[u][c] * v1f[c];
                } else if (pos >= 0) {
                    const T* kr = reinterpret_cast<const T*>(dsm) + (size_t)(pos % W) * D;
                    const T* vr = reinterpret_cast<const T*>(dsm + P.off_v) + (size_t)(pos % W) * D;
#pragma unroll
                    for (int c = 0; c < CPL; ++c) a += wk[u][c] * to_f(kr[lane + 32 * c]) + wv[u][c] * to_f(vr[lane + 32 * c]);
                }
                a = warp_sum(a);
                if (lane == 0) s_tap[t] = a;
            }
        }
        float m_loc = -INFINITY;
        if (wid == DT / 32 - 1) {
            float s = 0.f;
#pragma unroll
            for (int c = 0; c < CPL; ++c) s = fmaf(q1f[c], k1f[c], s);
            s = warp_sum(s) * scale;
            if (lane == 0) s_log[rows] = s;
            m_loc = s;
        }
        DPROF(3);
        // ---- logits of every cached row, masked, with the running max ---------------------------------------
        // Old ring row r holds the token at slot r; valid window rows are tokens n-W+1 .. n-1.  The popped row (slot)
        // stays in the sum iff it was accepted into the pool.  Old pool row m: valid iff m < cnt_old and m != dst.
        for (int r0 = 0; r0 < rows; r0 += 4 * RPP) {            // uniform trip count: the shuffles need every lane
            float sv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int row = r0 + u * RPP + rsub;
                float s0 = 0.f, s1 = 0.f;
                if (row < rows) {
                    float kf[EPV];
                    unpack<T>(Kc[(size_t)row * LPR + seg], kf);
#pragma unroll
                    for (int e = 0; e < EPV; e += 2) { s0 = fmaf(qf[e], kf[e], s0); s1 = fmaf(qf[e + 1], kf[e + 1], s1); }
                }
                sv[u] = s0 + s1;
            }
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) {
#pragma unroll
                for (int u = 0; u < 4; ++u) sv[u] += __shfl_xor_sync(0xffffffffu, sv[u], o);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int row = r0 + u * RPP + rsub;
                if (row < rows) {
                    bool ok;
                    if (row < W) ok = (n >= W) ? (row != slot || dst >= 0) : (row < n);
                    else ok = (row - W) < cnt_old && (row - W) != dst;
                    const float sl = ok ? sv[u] * scale : -INFINITY;
                    m_loc = fmaxf(m_loc, sl);
                    if (seg == 0) s_log[row] = sl;
                }
            }
        }
        m_loc = warp_max(m_loc);
        if (lane == 0) s_part[wid] = m_loc;
        // the popped row doubles as the new pool entry: keep it before the buffers are handed back
        uint4 mv = make_uint4(0, 0, 0, 0);
        if (tid < 2 * LPR) mv = (tid < LPR ? Kc : Vc)[(size_t)slot * LPR + (tid % LPR)];
        DPROF(4);
        __syncthreads();                                        // (A) every read of the key buffer is done
        DPROF(5);
        if (tid == 0 && bh + 1 < bh_end)
            bulk_load(sK, gblk + L.stride + L.off_k, P.kv_bytes, bar_k);
        float mx = s_part[0];
#pragma unroll
        for (int w2 = 1; w2 < DT / 32; ++w2) mx = fmaxf(mx, s_part[w2]);

        // ---- PV with the exponentials taken in place; the row sum rides along ------------------------------
        float acc[EPV], lsum = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) acc[e] = 0.f;
        for (int r0 = 0; r0 < rows; r0 += 4 * RPP) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int row = r0 + u * RPP + rsub;
                if (row < rows) {
                    const float pr = __expf(s_log[row] - mx);   // exp(-inf) = 0 for masked rows
                    if (pr != 0.f) {
                        float vf[EPV];
                        unpack<T>(Vc[(size_t)row * LPR + seg], vf);
#pragma unroll
                        for (int e = 0; e < EPV; ++e) acc[e] = fmaf(pr, vf[e], acc[e]);
                        if (seg == 0) lsum += pr;
                    }
                }
            }
        }
#pragma unroll
        for (int o = 16; o >= LPR; o >>= 1) {
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
        }
        lsum = warp_sum(lsum);
        if (lane < LPR) {
#pragma unroll
            for (int e = 0; e < EPV; ++e) s_red[wid][lane * EPV + e] = acc[e];
        }
        if (lane == 0) s_sum[wid] = lsum;
        DPROF(6);
        __syncthreads();                                        // (B) every read of the value buffer is done
        DPROF(7);
        if (tid == 0 && bh + 1 < bh_end) {
            bulk_load(sV, gblk + L.stride + L.off_v, P.kv_bytes, bar_v);
            bulk_load(sT + (tb ^ 1) * P.tail_bytes, gblk + L.stride + L.off_z, P.tail_bytes, bar_t0 + 8 * (tb ^ 1));
        }
        const float p_new = __expf(s_log[rows] - mx);
        float sum = p_new;
#pragma unroll
        for (int w2 = 0; w2 < DT / 32; ++w2) sum += s_sum[w2];
        if (tid < D) {
            float o = 0.f;
#pragma unroll
            for (int w2 = 0; w2 < DT / 32; ++w2) o += s_red[w2][tid];
            o = fmaf(p_new, v1_mine, o);
            o1[(size_t)bh * G * D + tid] = from_f<T>(o / sum);
        }
        if (tid == 0) lse1[(size_t)bh * G] = mx + logf(sum);

        // ---- write-back: only what changed goes to HBM -----------------------------------------------------
        uint4* Kw = reinterpret_cast<uint4*>(gblk + L.off_k);
        uint4* Vw = reinterpret_cast<uint4*>(gblk + L.off_v);
        float* zw = reinterpret_cast<float*>(gblk + L.off_z);
        int32_t* pw = reinterpret_cast<int32_t*>(gblk + L.off_pidx);
        int32_t* mw = reinterpret_cast<int32_t*>(gblk + L.off_meta);
        if (dst >= 0 && tid < 2 * LPR) (tid < LPR ? Kw : Vw)[(size_t)(W + dst) * LPR + (tid % LPR)] = mv;
        if (tid >= 64 && tid < 64 + 2 * LPR) {
            const int t2 = tid - 64;
            (t2 < LPR ? Kw : Vw)[(size_t)slot * LPR + (t2 % LPR)] = kv_new;
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
        DPROF(8);
        __syncthreads();                                        // (C) shared scratch is reused by the next head
        if (bh + 1 < bh_end) fetch_inputs(bh + 1);
        DPROF(9);
    }
}

// State after a T-token prompt.  One block per (b,h); the cache was zero-filled beforehand.
template <typename T>
__global__ void cache_init_kernel(unsigned char* __restrict__ cache, CacheLayout L, const T* __restrict__ k,
                                  const T* __restrict__ v, const float* __restrict__ z, const int32_t* __restrict__ idx,
                                  const int32_t* __restrict__ cnt, int Tlen, int D, int W, int R, int half)
{
    const int bh = blockIdx.x;
    unsigned char* blk = cache + L.header + (size_t)bh * L.stride;
    T* Kc = reinterpret_cast<T*>(blk + L.off_k);
    T* Vc = reinterpret_cast<T*>(blk + L.off_v);
    float* zc = reinterpret_cast<float*>(blk + L.off_z);
    int32_t* pidx = reinterpret_cast<int32_t*>(blk + L.off_pidx);
    int32_t* meta = reinterpret_cast<int32_t*>(blk + L.off_meta);
    const int n_ret = Tlen > 0 && R > 0 ? cnt[bh] : 0;
    const int lo = Tlen - W > 0 ? Tlen - W : 0;
    const int nwin = Tlen - lo;
    for (int e = threadIdx.x; e < (nwin + n_ret) * D; e += blockDim.x) {
        const int a = e / D, c = e % D;
        const int pos = a < nwin ? lo + a : idx[(size_t)bh * R + (a - nwin)];
        const int row = a < nwin ? pos % W : W + (a - nwin);
        const int cdst = L.swz ? ((((c >> 3) ^ (row & 7)) << 3) | (c & 7)) : c;   // swizzled layout: chunk c/8 moves
        Kc[(size_t)row * D + cdst] = k[((size_t)bh * Tlen + pos) * D + c];
        Vc[(size_t)row * D + cdst] = v[((size_t)bh * Tlen + pos) * D + c];
    }
    for (int a = threadIdx.x; a < W + R; a += blockDim.x) {
        float zz = -INFINITY;
        if (a < W) {
            // slot a holds the newest position congruent to a (mod W), if any
            if (a < nwin || Tlen >= W) {
                int pos = lo + ((a - lo % W) + W) % W;
                if (pos < Tlen && pos <= Tlen - 1 - half) zz = z[(size_t)bh * Tlen + pos];
            }
        } else if (a - W < n_ret) {
            const int pos = idx[(size_t)bh * R + (a - W)];
            zz = z[(size_t)bh * Tlen + pos];
            pidx[a - W] = pos;
        }
        zc[a] = zz;
    }
    if (threadIdx.x == 0) { meta[0] = Tlen; meta[1] = n_ret; meta[2] = 0; meta[3] = 0; }
}

}  // namespace

int decode_status_fetch_and_clear() { return status_fetch_and_clear(g_decode_status); }

int launch_cache_init(const Params& p, const void* k, const void* v, const float* z, const int32_t* idx,
                      const int32_t* cnt, void* cache, cudaStream_t st)
{
    const CacheLayout L = cache_layout(p.d, p.W, p.R, p.dtype);
    const size_t bytes = L.header + (size_t)p.B * p.H * L.stride;
    cudaError_t e = cudaMemsetAsync(cache, 0, bytes, st);
    if (e != cudaSuccess) return LTE_ERR_CUDA;
    if (p.dtype == LTE_BF16)
        cache_init_kernel<__nv_bfloat16><<<p.B * p.H, 256, 0, st>>>((unsigned char*)cache, L, (const __nv_bfloat16*)k,
                                                                    (const __nv_bfloat16*)v, z, idx, cnt, p.T, p.d, p.W,
                                                                    p.R, p.half);
    else
        cache_init_kernel<float><<<p.B * p.H, 256, 0, st>>>((unsigned char*)cache, L, (const float*)k, (const float*)v, z,
                                                            idx, cnt, p.T, p.d, p.W, p.R, p.half);
    return cuda_status(cudaGetLastError());
}

// ---- lazy scoring of the ring for scorers that do not run inside the step (the three-layer stack) -------------------
// The ring's rows in time order: row r of the copy is token base + r, base = max(n - W, 0); rows past the newest token are
// zero.  The scorer then runs over the copy as over a W-token sequence, and the logits whose receptive field lies inside
// the ring (or left of time 0) go back to the ring's logit slots: rows r >= half unless the ring starts at time 0, and
// r <= min(n, W) - 1 - half.
// With rotary tables (cos, sin [rope_len, D/2], half-split pairing: channels c and c + D/2 form a pair) the keys are
// rotated back to their un-rotated form on the way: the scorer consumes keys as they were before the position embedding,
// the cache holds them after it (Section 3.1.3, lazy scoring paragraph).  Row r is the token at position base + r.
template <typename T>
__global__ void ring_linearize_kernel(const unsigned char* __restrict__ cache, CacheLayout L, T* __restrict__ klin,
                                      T* __restrict__ vlin, int D, int W, const float* __restrict__ rope_cos,
                                      const float* __restrict__ rope_sin, int rope_len)
{
    const int bh = blockIdx.x;
    const unsigned char* blk = cache + L.header + (size_t)bh * L.stride;
    const T* Kc = reinterpret_cast<const T*>(blk + L.off_k);
    const T* Vc = reinterpret_cast<const T*>(blk + L.off_v);
    const int n = reinterpret_cast<const int32_t*>(blk + L.off_meta)[0];
    const int base = n > W ? n - W : 0, n_eff = n < W ? n : W;
    for (int e = threadIdx.x; e < W * D; e += blockDim.x) {
        const int r = e / D, c = e % D;
        T kx = from_f<T>(0.f), vx = from_f<T>(0.f);
        if (r < n_eff) {
            const int row = (base + r) % W;
            const int cs = L.swz ? ((((c >> 3) ^ (row & 7)) << 3) | (c & 7)) : c;
            kx = Kc[(size_t)row * D + cs]; vx = Vc[(size_t)row * D + cs];
            if (rope_cos) {
                const int pos = base + r, hd = D / 2;
                if (pos < rope_len) {
                    const int cp = c < hd ? c + hd : c - hd;       // the channel this one is paired with
                    const int cps = L.swz ? ((((cp >> 3) ^ (row & 7)) << 3) | (cp & 7)) : cp;
                    const float co = rope_cos[(size_t)pos * hd + (c % hd)], si = rope_sin[(size_t)pos * hd + (c % hd)];
                    const float a = to_f(kx), b = to_f(Kc[(size_t)row * D + cps]);
                    // inverse rotation: (x1, x2) -> (x1 cos + x2 sin, x2 cos - x1 sin)
                    kx = from_f<T>(c < hd ? a * co + b * si : a * co - b * si);
                } else if (c == 0) {
                    atomicExch(&g_decode_status.code, 32);              // the tables do not reach this position: key left rotated
                }
            }
        }
        klin[((size_t)bh * W + r) * D + c] = kx;
        vlin[((size_t)bh * W + r) * D + c] = vx;
    }
}

__global__ void ring_scatter_z_kernel(unsigned char* __restrict__ cache, CacheLayout L, const float* __restrict__ zlin, int W,
                                      int half)
{
    const int bh = blockIdx.x;
    unsigned char* blk = cache + L.header + (size_t)bh * L.stride;
    float* zc = reinterpret_cast<float*>(blk + L.off_z);
    const int n = reinterpret_cast<const int32_t*>(blk + L.off_meta)[0];
    const int base = n > W ? n - W : 0, n_eff = n < W ? n : W;
    const int r_lo = base > 0 ? half : 0, r_hi = n_eff - 1 - half;
    for (int r = r_lo + threadIdx.x; r <= r_hi; r += blockDim.x) zc[(base + r) % W] = zlin[(size_t)bh * W + r];
}

int launch_ring_linearize(const Params& p, const void* cache, void* klin, void* vlin, const float* rope_cos, const float* rope_sin,
                          int rope_len, cudaStream_t st)
{
    const CacheLayout L = cache_layout(p.d, p.W, p.R, p.dtype);
    if (p.dtype == LTE_BF16)
        ring_linearize_kernel<__nv_bfloat16><<<p.B * p.H, 256, 0, st>>>((const unsigned char*)cache, L, (__nv_bfloat16*)klin,
                                                                        (__nv_bfloat16*)vlin, p.d, p.W, rope_cos, rope_sin, rope_len);
    else
        ring_linearize_kernel<float><<<p.B * p.H, 256, 0, st>>>((const unsigned char*)cache, L, (float*)klin, (float*)vlin, p.d, p.W,
                                                                rope_cos, rope_sin, rope_len);
    return cuda_status(cudaGetLastError());
}

int launch_ring_scatter_z(const Params& p, void* cache, const float* zlin, cudaStream_t st)
{
    const CacheLayout L = cache_layout(p.d, p.W, p.R, p.dtype);
    ring_scatter_z_kernel<<<p.B * p.H, 128, 0, st>>>((unsigned char*)cache, L, zlin, p.W, p.half);
    return cuda_status(cudaGetLastError());
}

// ---- grouped-query attention -----------------------------------------------------------------------------------------
// With G > 1 query heads per key/value head the cache block is read once per step: the head's thread block first applies
// the replacement rule, scores the newest complete token and writes the new key/value into the ring (a handful of rows),
// then serves all G query heads over the updated block (the attend kernel below).
// The update of one key/value head's block by the DTU threads of a thread block (every thread of the block calls it; it
// ends with the block's writes issued, not yet ordered: the caller synchronises).
template <typename T, int D, int DTU>
__device__ __forceinline__ void cache_update_block(unsigned char* __restrict__ cache, const CacheLayout& L, int bh,
                                                   const T* __restrict__ k1, const T* __restrict__ v1,
                                                   const float* __restrict__ cw, const float* __restrict__ cbias, int H,
                                                   int W, int R, int sink, int K, float zthr)
{
    constexpr int CPL = D / 32, NWU = DTU / 32, PIECES = D * (int)sizeof(T) / 16;
    __shared__ float s_tap[kMaxTaps];
    __shared__ float s_wz[NWU];
    __shared__ int s_wpos[NWU], s_wslot[NWU];
    const int h = bh % H, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    unsigned char* blk = cache + L.header + (size_t)bh * L.stride;
    T* Kc = reinterpret_cast<T*>(blk + L.off_k);
    T* Vc = reinterpret_cast<T*>(blk + L.off_v);
    float* zc = reinterpret_cast<float*>(blk + L.off_z);
    int32_t* pidx = reinterpret_cast<int32_t*>(blk + L.off_pidx);
    int32_t* meta = reinterpret_cast<int32_t*>(blk + L.off_meta);
    const int n = meta[0], cnt_old = meta[1];
    const int slot = n % W, p = n - W, half = K / 2;
    // element ch of row r (the swizzled layout permutes the 16-byte pieces of a row)
    auto pos_of = [&](int r, int ch) { return L.swz ? ((((ch >> 3) ^ (r & 7)) << 3) | (ch & 7)) : ch; };

    // ---- the token leaving the window is offered to the pool (same rule as the step kernels) ----
    int dst = -1, cnt_new = cnt_old;
    float zp = 0.f;
    if (p >= 0 && R > 0) {
        zp = zc[slot];
        const bool is_sink = p < sink;
        if (is_sink || zp > zthr) {
            if (cnt_old < R) { dst = cnt_old; cnt_new = cnt_old + 1; }
            else if (!is_sink) {
                // worst entry: lowest logit, the youngest among equals, never a sink entry
                float wz = INFINITY; int wpos = -1, wslot = -1;
                for (int m = tid; m < cnt_old; m += DTU) {
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
                if (lane == 0) { s_wz[wid] = wz; s_wpos[wid] = wpos; s_wslot[wid] = wslot; }
                __syncthreads();
                wz = s_wz[0]; wpos = s_wpos[0]; wslot = s_wslot[0];
#pragma unroll
                for (int w2 = 1; w2 < NWU; ++w2) {
                    const float oz = s_wz[w2]; const int op = s_wpos[w2], os = s_wslot[w2];
                    if (os >= 0 && (wslot < 0 || oz < wz || (oz == wz && op > wpos))) { wz = oz; wpos = op; wslot = os; }
                }
                if (wslot >= 0 && zp > wz) dst = wslot;
            }
        }
    }
    // ---- logit of the newest token whose receptive field is complete (K = 0: scored outside the step) ----
    const int jsc = K > 0 ? n - half : -1;
    if (jsc >= 0) {
        for (int t = wid; t < K; t += NWU) {
            const int pos = jsc + t - half;
            float a = 0.f;
            if (pos >= 0) {
#pragma unroll
                for (int c = 0; c < CPL; ++c) {
                    const int ch = lane + 32 * c;
                    const float wk = cw[((size_t)h * K + t) * 2 * D + ch], wv = cw[((size_t)h * K + t) * 2 * D + D + ch];
                    float kx, vx;
                    if (pos == n) { kx = to_f(k1[(size_t)bh * D + ch]); vx = to_f(v1[(size_t)bh * D + ch]); }
                    else { const int r = pos % W; kx = to_f(Kc[(size_t)r * D + pos_of(r, ch)]); vx = to_f(Vc[(size_t)r * D + pos_of(r, ch)]); }
                    a += wk * kx + wv * vx;
                }
            }
            a = warp_sum(a);
            if (lane == 0) s_tap[t] = a;
        }
    }
    // ---- moves: the popped row into its pool row, the new key/value into the ring slot ----
    uint4 mv = make_uint4(0, 0, 0, 0), nw = mv;
    const bool mover = tid < 2 * PIECES;
    const int pc = tid % PIECES;                               // logical 16-byte piece of the row
    if (mover) {
        const uint4* src = reinterpret_cast<const uint4*>(tid < PIECES ? Kc : Vc);
        mv = src[(size_t)slot * PIECES + (L.swz ? (pc ^ (slot & 7)) : pc)];
        nw = reinterpret_cast<const uint4*>((tid < PIECES ? k1 : v1) + (size_t)bh * D)[pc];
    }
    __syncthreads();                                           // the ring rows the taps read are still the old ones up to here
    if (mover) {
        uint4* dstp = reinterpret_cast<uint4*>(tid < PIECES ? Kc : Vc);
        if (dst >= 0) dstp[(size_t)(W + dst) * PIECES + (L.swz ? (pc ^ ((W + dst) & 7)) : pc)] = mv;
        dstp[(size_t)slot * PIECES + (L.swz ? (pc ^ (slot & 7)) : pc)] = nw;
    }
    if (tid == 0) {
        if (dst >= 0) { zc[W + dst] = zp; pidx[dst] = p; }
        float znew = -INFINITY;
        if (jsc >= 0) {
            znew = cbias ? cbias[h] : 0.f;
            for (int t = 0; t < K; ++t) znew += s_tap[t];
        }
        zc[slot] = -INFINITY;
        if (jsc >= 0) zc[jsc % W] = znew;
        meta[0] = n + 1;
        meta[1] = cnt_new;
    }
}

// The attend kernel: query heads g_first .. G-1 of a key/value head over its block (ring rows of the min(n, W) newest
// tokens, cnt pool rows), after the update.  One block (or a cluster of blocks) per key/value head, up to ATT_Q query heads
// per pass.  Rows are spread as in the step kernels: LPR lanes share a row, each with one 16-byte piece of it, so a warp's
// load covers whole consecutive rows; eight rows per thread are in flight.  Logits: partial dots per lane against the
// lane's slice of every query, reduced over the LPR lanes by shuffles; block maxima and sums per query head; value rows
// the same way, weighted per query head in registers, reduced over lanes sharing a slice and then over the warps.
constexpr int ATT_Q = 4;
template <typename T, int D>
__global__ void __launch_bounds__(DT) decode_attend_kernel(unsigned char* __restrict__ cache, CacheLayout L,
                                                           const T* __restrict__ q1, T* __restrict__ o1,
                                                           float* __restrict__ lse1, int W, int G, float scale, int g_first,
                                                           const T* __restrict__ k1, const T* __restrict__ v1,
                                                           const float* __restrict__ cw, const float* __restrict__ cbias, int H,
                                                           int R, int sink, int K, float zthr)
{
    constexpr int EPV = V16<T>::N;                             // elements per 16-byte piece
    constexpr int LPR = D / EPV;                               // lanes per row
    constexpr int RPP = DT / LPR;                              // rows per pass of the block
    constexpr int NW = DT / 32, UNR = 8;
    extern __shared__ float att_sm[];                          // logits [ATT_Q][rows], then partial outputs [NW][ATT_Q][D]
    __shared__ float s_red[NW][ATT_Q];
    __shared__ float s_mx[ATT_Q], s_sum[ATT_Q];
    __shared__ float s_fin[ATT_Q][D];                          // this block's unnormalised outputs (read by the cluster's first block)
    // A thread-block cluster shares one key/value head: block `rank` of `nsplit` takes a contiguous share of the rows,
    // and the first block combines the partial maxima, sums and outputs through distributed shared memory.
    cg::cluster_group cluster = cg::this_cluster();
    const int nsplit = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const int bh = blockIdx.x / nsplit, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int seg = tid % LPR, rsub = tid / LPR;
    // the step's cache update first (k1 != NULL), by the head's (first) block: a handful of rows, then everybody reads the
    // updated block
    if (k1 != nullptr) {
        if (rank == 0) {
            cache_update_block<T, D, DT>(cache, L, bh, k1, v1, cw, cbias, H, W, R, sink, K, zthr);
            __threadfence();
        }
        if (nsplit > 1) cluster.sync(); else __syncthreads();
    }
    const unsigned char* blk = cache + L.header + (size_t)bh * L.stride;
    const uint4* Kc = reinterpret_cast<const uint4*>(blk + L.off_k);
    const uint4* Vc = reinterpret_cast<const uint4*>(blk + L.off_v);
    const int32_t* meta = reinterpret_cast<const int32_t*>(blk + L.off_meta);
    const int n = meta[0], cnt = meta[1];
    const int n_ring = n < W ? n : W, rows_all = n_ring + cnt;
    const int share = (rows_all + nsplit - 1) / nsplit;
    const int a_lo = min(rank * share, rows_all), rows = min(a_lo + share, rows_all) - a_lo;   // this block's rows: a_lo + [0, rows)
    float* s_log = att_sm;
    float* s_out = att_sm + (size_t)ATT_Q * rows;
    // this thread's piece of list entry a: cache row (ring rows first, then pool rows) and the piece's place in it (the
    // swizzled layout permutes the pieces of a row)
    auto piece_of = [&](int a) {
        const int r = a_lo + a < n_ring ? a_lo + a : W + (a_lo + a - n_ring);
        return (size_t)r * LPR + (L.swz ? (seg ^ (r & 7)) : seg);
    };
    for (int g0 = g_first; g0 < G; g0 += ATT_Q) {
        const int nq = G - g0 < ATT_Q ? G - g0 : ATT_Q;
        float qv[ATT_Q][EPV];                                  // this lane's slice of the pass's queries, pre-scaled
#pragma unroll
        for (int u = 0; u < ATT_Q; ++u)
#pragma unroll
            for (int e = 0; e < EPV; ++e)
                qv[u][e] = u < nq ? to_f(q1[((size_t)bh * G + g0 + u) * D + seg * EPV + e]) * scale : 0.f;
        // ---- logits ----
        float mx[ATT_Q];
#pragma unroll
        for (int u = 0; u < ATT_Q; ++u) mx[u] = -INFINITY;
        for (int a0 = 0; a0 < rows; a0 += UNR * RPP) {         // uniform trip count: the shuffles need every lane
            uint4 raw[UNR];
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                const int a = a0 + j * RPP + rsub;
                raw[j] = a < rows ? Kc[piece_of(a)] : make_uint4(0, 0, 0, 0);
            }
            float dot[UNR][ATT_Q];
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                float kf[EPV];
                unpack<T>(raw[j], kf);
#pragma unroll
                for (int u = 0; u < ATT_Q; ++u) {
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int e = 0; e < EPV; e += 2) { s0 = fmaf(qv[u][e], kf[e], s0); s1 = fmaf(qv[u][e + 1], kf[e + 1], s1); }
                    dot[j][u] = s0 + s1;
                }
            }
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1)
#pragma unroll
                for (int j = 0; j < UNR; ++j)
#pragma unroll
                    for (int u = 0; u < ATT_Q; ++u) dot[j][u] += __shfl_xor_sync(0xffffffffu, dot[j][u], o);
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                const int a = a0 + j * RPP + rsub;
                if (a < rows) {
#pragma unroll
                    for (int u = 0; u < ATT_Q; ++u) {
                        mx[u] = fmaxf(mx[u], dot[j][u]);
                        if (seg == u % LPR) s_log[(size_t)u * rows + a] = dot[j][u];   // (the LPR lanes hold the same sums: spread the stores)
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < ATT_Q; ++u) mx[u] = warp_max(mx[u]);
        if (lane == 0)
#pragma unroll
            for (int u = 0; u < ATT_Q; ++u) s_red[wid][u] = mx[u];
        __syncthreads();
        if (tid < ATT_Q) {
            float m = -INFINITY;
            for (int w2 = 0; w2 < NW; ++w2) m = fmaxf(m, s_red[w2][tid]);
            s_mx[tid] = m;
        }
        __syncthreads();
        // ---- probabilities in place, their sums ----
        float ps[ATT_Q];
#pragma unroll
        for (int u = 0; u < ATT_Q; ++u) {
            ps[u] = 0.f;
            const float m = s_mx[u];
            for (int a = tid; a < rows; a += DT) {
                const float pj = __expf(s_log[(size_t)u * rows + a] - m);
                s_log[(size_t)u * rows + a] = pj;
                ps[u] += pj;
            }
            ps[u] = warp_sum(ps[u]);
        }
        if (lane == 0)
#pragma unroll
            for (int u = 0; u < ATT_Q; ++u) s_red[wid][u] = ps[u];
        __syncthreads();
        if (tid < ATT_Q) {
            float t = 0.f;
            for (int w2 = 0; w2 < NW; ++w2) t += s_red[w2][tid];
            s_sum[tid] = t;
        }
        // ---- weighted value rows ----
        float acc[ATT_Q][EPV];
#pragma unroll
        for (int u = 0; u < ATT_Q; ++u)
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[u][e] = 0.f;
        for (int a0 = 0; a0 < rows; a0 += UNR * RPP) {
            uint4 raw[UNR];
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                const int a = a0 + j * RPP + rsub;
                raw[j] = a < rows ? Vc[piece_of(a)] : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                const int a = min(a0 + j * RPP + rsub, rows - 1);   // (rows past the end carry zero values)
                float vf[EPV];
                unpack<T>(raw[j], vf);
#pragma unroll
                for (int u = 0; u < ATT_Q; ++u) {
                    const float pj = s_log[(size_t)u * rows + a];
#pragma unroll
                    for (int e = 0; e < EPV; ++e) acc[u][e] = fmaf(pj, vf[e], acc[u][e]);
                }
            }
        }
        // lanes that share a slice of the row (same seg) add up, then the warps
#pragma unroll
        for (int o = 16; o >= LPR; o >>= 1)
#pragma unroll
            for (int u = 0; u < ATT_Q; ++u)
#pragma unroll
                for (int e = 0; e < EPV; ++e) acc[u][e] += __shfl_xor_sync(0xffffffffu, acc[u][e], o);
        if (lane < LPR) {
#pragma unroll
            for (int u = 0; u < ATT_Q; ++u)
#pragma unroll
                for (int e = 0; e < EPV; ++e) s_out[((size_t)wid * ATT_Q + u) * D + lane * EPV + e] = acc[u][e];
        }
        __syncthreads();
        for (int e = tid; e < nq * D; e += DT) {
            const int u = e / D, ch = e - u * D;
            float t = 0.f;
            for (int w2 = 0; w2 < NW; ++w2) t += s_out[((size_t)w2 * ATT_Q + u) * D + ch];
            s_fin[u][ch] = t;
        }
        cluster.sync();                                        // every block's partial results are in its shared memory
        if (rank == 0) {
            for (int e = tid; e < nq * D; e += DT) {
                const int u = e / D, ch = e - u * D;
                float m = -INFINITY;
                for (int r2 = 0; r2 < nsplit; ++r2) m = fmaxf(m, *cluster.map_shared_rank(&s_mx[u], r2));
                float tot = 0.f, acc2 = 0.f;
                for (int r2 = 0; r2 < nsplit; ++r2) {
                    const float f = expf(*cluster.map_shared_rank(&s_mx[u], r2) - m);   // a block without rows: exp(-inf) = 0
                    tot = fmaf(f, *cluster.map_shared_rank(&s_sum[u], r2), tot);
                    acc2 = fmaf(f, *cluster.map_shared_rank(&s_fin[u][ch], r2), acc2);
                }
                o1[((size_t)bh * G + g0 + u) * D + ch] = from_f<T>(acc2 / tot);
                if (ch == 0) lse1[(size_t)bh * G + g0 + u] = m + logf(tot);
            }
        }
        cluster.sync();                                        // the partial results may be overwritten by the next pass (or the block may exit)
    }
}

static int launch_decode_step(const Params& p, void* cache, const void* q1, const void* k1, const void* v1, void* o1, float* lse1,
                              cudaStream_t st)
{
    if (p.W + p.R > MAX_ROWS) return LTE_ERR_UNSUPPORTED;
    const CacheLayout L = cache_layout(p.d, p.W, p.R, p.dtype);
    if (L.swz) return launch_decode_tc(p, cache, q1, k1, v1, o1, lse1, st);   // bf16, d = 64, W+R <= 256: tensor-core kernel
    const BulkSmem bp = bulk_smem_plan(L, p.W, p.R);
    const size_t bulk_smem = bp.total;
    const bool bulk = bulk_smem <= 73 * 1024 && p.K <= 2 * (DT / 32);   // three blocks per SM still fit
    int n_sm = 0;
    if (int e = device_sm_count(&n_sm)) return e;
    // persistent grid: every CTA walks `per_cta` consecutive heads; all CTAs are resident (3 per SM)
    const int BH = p.B * p.H;
    const int per_cta = bulk ? (BH + 3 * n_sm - 1) / (3 * n_sm) : 1;
    const int n_cta = bulk ? (BH + per_cta - 1) / per_cta : BH;
#define LTE_BULK(T, D)                                                                                            \
    do {                                                                                                          \
        static PerDeviceOnce attr;                                                                                \
        if (int e = attr.run([] { return cudaFuncSetAttribute(decode_bulk_kernel<T, D>,                           \
                cudaFuncAttributeMaxDynamicSharedMemorySize, 73 * 1024); })) return e;                            \
        decode_bulk_kernel<T, D><<<n_cta, DT, bulk_smem, st>>>((unsigned char*)cache, L, (const T*)q1,             \
            (const T*)k1, (const T*)v1, (T*)o1, lse1, p.w, p.bias, BH, per_cta, p.H, p.W, p.R, p.sink, p.K,        \
            p.zthr, p.scale, p.G);                                                                                     \
    } while (0)
    if (bulk) {
        if (p.dtype == LTE_BF16) {
            switch (p.d) {
                case 32: LTE_BULK(__nv_bfloat16, 32); break;
                case 64: LTE_BULK(__nv_bfloat16, 64); break;
                case 128: LTE_BULK(__nv_bfloat16, 128); break;
                default: return LTE_ERR_UNSUPPORTED;
            }
        } else {
            switch (p.d) {
                case 32: LTE_BULK(float, 32); break;
                case 64: LTE_BULK(float, 64); break;
                case 128: LTE_BULK(float, 128); break;
                default: return LTE_ERR_UNSUPPORTED;
            }
        }
        return cuda_status(cudaGetLastError());
    }
#undef LTE_BULK
#define LTE_GO(T, D)                                                                                              \
    decode_kernel<T, D><<<p.B * p.H, DT, 0, st>>>((unsigned char*)cache, L, (const T*)q1, (const T*)k1, (const T*)v1, \
                                                  (T*)o1, lse1, p.w, p.bias, p.H, p.W, p.R, p.sink, p.K, p.zthr,   \
                                                  p.scale, p.G)
    if (p.dtype == LTE_BF16) {
        switch (p.d) {
            case 32: LTE_GO(__nv_bfloat16, 32); break;
            case 64: LTE_GO(__nv_bfloat16, 64); break;
            case 128: LTE_GO(__nv_bfloat16, 128); break;
            default: return LTE_ERR_UNSUPPORTED;
        }
    } else {
        switch (p.d) {
            case 32: LTE_GO(float, 32); break;
            case 64: LTE_GO(float, 64); break;
            case 128: LTE_GO(float, 128); break;
            default: return LTE_ERR_UNSUPPORTED;
        }
    }
#undef LTE_GO
    return cuda_status(cudaGetLastError());
}

int launch_decode(const Params& p, void* cache, const void* q1, const void* k1, const void* v1, void* o1, float* lse1,
                  cudaStream_t st)
{
    Params ps = p;
    if (p.stack) ps.K = 0;                               // the stack is scored outside the step (lte_cache_score)
    if (p.G <= 1) return launch_decode_step(ps, cache, q1, k1, v1, o1, lse1, st);
    // grouped queries: one kernel updates the head's cache block and then serves all query heads of the group from it
    if (p.W + p.R > MAX_ROWS) return LTE_ERR_UNSUPPORTED;
    const CacheLayout L = cache_layout(p.d, p.W, p.R, p.dtype);
    const size_t att_smem = sizeof(float) * ((size_t)ATT_Q * (p.W + p.R) + (size_t)(DT / 32) * ATT_Q * p.d);
    // blocks per key/value head (a cluster): more than one only while there are fewer blocks than SMs and a share keeps 256 rows
    // (with 256 heads of 1280 rows, two blocks per head measured 41 us per step against 29 us for one)
    int n_sm_att = 0;
    if (int e = device_sm_count(&n_sm_att)) return e;
    int nsplit = 1;
    while (nsplit < 8 && p.B * p.H * nsplit < n_sm_att && (p.W + p.R) / (2 * nsplit) >= 256) nsplit *= 2;
    cudaLaunchConfig_t acfg = {};
    acfg.gridDim = dim3(p.B * p.H * nsplit); acfg.blockDim = dim3(DT); acfg.dynamicSmemBytes = att_smem; acfg.stream = st;
    cudaLaunchAttribute aattr[1];
    aattr[0].id = cudaLaunchAttributeClusterDimension;
    aattr[0].val.clusterDim.x = nsplit; aattr[0].val.clusterDim.y = 1; aattr[0].val.clusterDim.z = 1;
    acfg.attrs = aattr; acfg.numAttrs = 1;
#define LTE_ATT(T, D)                                                                                                  \
    do {                                                                                                               \
        static PerDeviceOnce attr;                                                                                     \
        if (int e = attr.run([] { return cudaFuncSetAttribute(decode_attend_kernel<T, D>,                              \
                cudaFuncAttributeMaxDynamicSharedMemorySize,                                                           \
                (int)(sizeof(float) * ((size_t)ATT_Q * MAX_ROWS + (DT / 32) * ATT_Q * 128))); })) return e;            \
        if (cudaLaunchKernelEx(&acfg, decode_attend_kernel<T, D>, (unsigned char*)cache, L, (const T*)q1, (T*)o1, lse1,        \
                               p.W, p.G, p.scale, 0, (const T*)k1, (const T*)v1, p.w, p.bias, p.H, p.R, p.sink, ps.K,    \
                               p.zthr) != cudaSuccess) return LTE_ERR_CUDA;                                             \
    } while (0)
    if (p.dtype == LTE_BF16) {
        switch (p.d) {
            case 32: LTE_ATT(__nv_bfloat16, 32); break;
            case 64: LTE_ATT(__nv_bfloat16, 64); break;
            case 128: LTE_ATT(__nv_bfloat16, 128); break;
            default: return LTE_ERR_UNSUPPORTED;
        }
    } else {
        switch (p.d) {
            case 32: LTE_ATT(float, 32); break;
            case 64: LTE_ATT(float, 64); break;
            case 128: LTE_ATT(float, 128); break;
            default: return LTE_ERR_UNSUPPORTED;
        }
    }
#undef LTE_ATT
    return cuda_status(cudaGetLastError());
}

}  // namespace lte

#ifdef LTE_PROFILE
extern "C" int lte_dprof_read(long long* out)
{
    return cudaMemcpyFromSymbol(out, lte::g_dprof, sizeof(long long) * 64) == cudaSuccess ? 0 : -1;
}
#endif
