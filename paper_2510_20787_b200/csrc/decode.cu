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
#include "common.cuh"

namespace lte {
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
                                                    int K, float zthr, float scale)
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
        uint4 u = *reinterpret_cast<const uint4*>(q1 + (size_t)bh * D + seg * EPV);
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
        for (int c = lane; c < D; c += 32) s = fmaf(to_f(q1[(size_t)bh * D + c]) * scale, to_f(k1[(size_t)bh * D + c]), s);
        s = warp_sum(s);
        if (lane == 0) s_log[rows] = s;
    }
    __syncthreads();

    const int n = s_dec[0], cnt_old = s_dec[1], dst = s_dec[2], cnt_new = s_dec[3];
    const int slot = n % W;

    // ---- scorer for token j = n - half, from the old ring rows and the incoming row -------------
    const int jsc = n - half;
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
        o1[(size_t)bh * D + tid] = from_f<T>(o * inv);
    }
    if (tid == 0) lse1[bh] = mx + logf(sum);

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
        Kc[(size_t)row * D + c] = k[((size_t)bh * Tlen + pos) * D + c];
        Vc[(size_t)row * D + c] = v[((size_t)bh * Tlen + pos) * D + c];
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

int launch_decode(const Params& p, void* cache, const void* q1, const void* k1, const void* v1, void* o1, float* lse1,
                  cudaStream_t st)
{
    if (p.W + p.R > MAX_ROWS) return LTE_ERR_UNSUPPORTED;
    const CacheLayout L = cache_layout(p.d, p.W, p.R, p.dtype);
#define LTE_GO(T, D)                                                                                              \
    decode_kernel<T, D><<<p.B * p.H, DT, 0, st>>>((unsigned char*)cache, L, (const T*)q1, (const T*)k1, (const T*)v1, \
                                                  (T*)o1, lse1, p.w, p.bias, p.H, p.W, p.R, p.sink, p.K, p.zthr,   \
                                                  p.scale)
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

}  // namespace lte
