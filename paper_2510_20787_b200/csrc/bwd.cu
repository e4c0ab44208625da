// Backward of the LTE prefill attention with the straight-through surrogate (Section 3.1.2, Eq. 6, Eq. 7).
//
// Gather form, no floating-point atomics, so the result is deterministic:
//   dq kernel   one warp per query i: delta_i = <dO_i, o_i>, then over A_i (visible retained prefix + window)
//               P_ij = exp(scale q_i.k_j - lse_i), dS_ij = P_ij (<dO_i, v_j> - delta_i), dq_i = scale sum_j dS_ij k_j.
//   dkv kernel  one warp per key j: over the queries that see j (the W window queries j..j+W-1 and, if j is in the
//               retained list, every query >= j+W): dv_j = sum_i P_ij dO_i, dk_j = scale sum_i dS_ij q_i; then
//               Eq. 6: dr_j = <v_j, dv_j> (+ lambda_h 1[z_j > zthr]), dz_j = dr_j r_j (1 - r_j) for scored tokens.
//   conv kernels  dw, dbias as per-(b, chunk) partial sums reduced in a fixed order; with the input-gradient flag
//               the scorer's share sum_t dz[p-t+half] w[h,t,c] is added to the fp32 dk, dv before the one rounding.
// Workspace: delta, dz [B,H,T] fp32; dw/dbias partials; fp32 dk, dv [B,H,T,d] when the flag is set.
#include "common.cuh"
#include "tc_common.cuh"

namespace lte {

int launch_bwd_dq_tc(const Params& p, const void* q, const void* k, const void* v, const void* o, const float* lse,
                     const void* dO, const int32_t* idx, const int32_t* cnt, void* dq, float* delta, cudaStream_t st);

size_t bwd_tc_ret_bytes(const Params& p);
int launch_bwd_dkv_tc(const Params& p, const void* q, const void* k, const void* v, const float* lse, const void* dO,
                      const float* delta, const float* z, const int32_t* idx, const int32_t* cnt, const float* lambda,
                      void* dk, void* dv, float* dk32, float* dv32, float* dz, void* ret_ws, bool f32out, bool merge_here,
                      cudaStream_t st);

namespace {

constexpr int CHUNK = 256;     // positions per conv-gradient partial

template <typename T, int D>
__global__ void __launch_bounds__(128) bwd_dq_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                     const T* __restrict__ v, const T* __restrict__ o,
                                                     const T* __restrict__ dO, const float* __restrict__ lse,
                                                     const int32_t* __restrict__ idx, const int32_t* __restrict__ cnt,
                                                     T* __restrict__ dq, float* __restrict__ delta, int Tlen, int W,
                                                     int R, float scale, int G)
{
    constexpr int C = D / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * 4 + warp;
    const int bh = blockIdx.y, bhk = bh / G;                   // query head; its key/value head
    if (i >= Tlen) return;
    const size_t base = (size_t)bh * Tlen * D, kbase = (size_t)bhk * Tlen * D;
    float qv[C], gv[C], acc[C];
    float dl = 0.f;
#pragma unroll
    for (int c = 0; c < C; ++c) {
        const size_t e = base + (size_t)i * D + lane + 32 * c;
        qv[c] = to_f(q[e]) * scale; gv[c] = to_f(dO[e]); acc[c] = 0.f;
        dl = fmaf(gv[c], to_f(o[e]), dl);
    }
    dl = warp_sum(dl);
    if (lane == 0) delta[(size_t)bh * Tlen + i] = dl;
    const float li = lse[(size_t)bh * Tlen + i];
    const int32_t* id = idx + (size_t)bhk * R;
    const int n_ret = cnt[bhk];
    const int lo = i - W + 1 > 0 ? i - W + 1 : 0;
    int nvis = 0;
    for (int m0 = 0; m0 < n_ret; m0 += 32) {
        int e = m0 + lane < n_ret ? id[m0 + lane] : 0x7fffffff;
        unsigned b = __ballot_sync(0xffffffffu, e <= i - W);
        nvis += __popc(b);
        if (b != 0xffffffffu) break;
    }
    const int total = nvis + (i - lo + 1);
    for (int a = 0; a < total; ++a) {
        const int j = a < nvis ? id[a] : lo + (a - nvis);
        const T* kr = k + kbase + (size_t)j * D;
        const T* vr = v + kbase + (size_t)j * D;
        float s = 0.f, dp = 0.f, kk[C];
#pragma unroll
        for (int c = 0; c < C; ++c) {
            kk[c] = to_f(kr[lane + 32 * c]);
            s = fmaf(qv[c], kk[c], s);
            dp = fmaf(gv[c], to_f(vr[lane + 32 * c]), dp);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            s += __shfl_xor_sync(0xffffffffu, s, off);
            dp += __shfl_xor_sync(0xffffffffu, dp, off);
        }
        const float ds = expf(s - li) * (dp - dl);
#pragma unroll
        for (int c = 0; c < C; ++c) acc[c] = fmaf(ds, kk[c], acc[c]);
    }
#pragma unroll
    for (int c = 0; c < C; ++c) dq[base + (size_t)i * D + lane + 32 * c] = from_f<T>(acc[c] * scale);
}

template <typename T, int D, bool F32OUT>
__global__ void __launch_bounds__(128) bwd_dkv_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                      const T* __restrict__ v, const T* __restrict__ dO,
                                                      const float* __restrict__ lse, const float* __restrict__ delta,
                                                      const float* __restrict__ z, const int32_t* __restrict__ idx,
                                                      const int32_t* __restrict__ cnt, const float* __restrict__ lambda,
                                                      T* __restrict__ dk, T* __restrict__ dv, float* __restrict__ dk32,
                                                      float* __restrict__ dv32, float* __restrict__ dz, int H, int Tlen,
                                                      int W, int R, int half, float zthr, float scale, int G)
{
    constexpr int C = D / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = blockIdx.x * 4 + warp;
    const int bh = blockIdx.y;
    if (j >= Tlen) return;
    const size_t base = (size_t)bh * Tlen * D;
    float kv[C], vv[C], ak[C], av[C];
#pragma unroll
    for (int c = 0; c < C; ++c) {
        const size_t e = base + (size_t)j * D + lane + 32 * c;
        kv[c] = to_f(k[e]) * scale; vv[c] = to_f(v[e]); ak[c] = 0.f; av[c] = 0.f;
    }
    // is j in the retained list? (idx ascending: binary search, uniform across the warp)
    bool kept = false;
    {
        const int32_t* id = idx + (size_t)bh * R;
        int lo = 0, hi = cnt[bh];
        while (lo < hi) { int mid = (lo + hi) >> 1; if (id[mid] < j) lo = mid + 1; else hi = mid; }
        kept = lo < cnt[bh] && id[lo] == j;
    }
    const int iend = kept ? Tlen - 1 : (j + W - 1 < Tlen - 1 ? j + W - 1 : Tlen - 1);
    for (int gi = 0; gi < G * (iend - j + 1); ++gi) {          // the group's query heads in turn, each over its queries
        const int g = gi / (iend - j + 1), i = j + gi % (iend - j + 1);
        const size_t qbase = ((size_t)bh * G + g) * Tlen;
        const T* qr = q + (qbase + i) * D;
        const T* gr = dO + (qbase + i) * D;
        float s = 0.f, dp = 0.f, qq[C], gg[C];
#pragma unroll
        for (int c = 0; c < C; ++c) {
            qq[c] = to_f(qr[lane + 32 * c]); gg[c] = to_f(gr[lane + 32 * c]);
            s = fmaf(qq[c], kv[c], s);
            dp = fmaf(gg[c], vv[c], dp);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            s += __shfl_xor_sync(0xffffffffu, s, off);
            dp += __shfl_xor_sync(0xffffffffu, dp, off);
        }
        const float p = expf(s - lse[qbase + i]);
        const float ds = p * (dp - delta[qbase + i]);
#pragma unroll
        for (int c = 0; c < C; ++c) { av[c] = fmaf(p, gg[c], av[c]); ak[c] = fmaf(ds, qq[c], ak[c]); }
    }
    // Eq. 6 on the attention-only dV; scored tokens only
    float dr = 0.f;
#pragma unroll
    for (int c = 0; c < C; ++c) dr = fmaf(vv[c], av[c], dr);
    dr = warp_sum(dr);
    if (lane == 0) {
        float g = 0.f;
        if (j + half <= Tlen - 1) {
            const float zz = z[(size_t)bh * Tlen + j];
            const float r = 1.f / (1.f + expf(-zz));
            if (lambda && zz > zthr) dr += lambda[bh % H];
            g = dr * r * (1.f - r);
        }
        dz[(size_t)bh * Tlen + j] = g;
    }
#pragma unroll
    for (int c = 0; c < C; ++c) {
        const size_t e = base + (size_t)j * D + lane + 32 * c;
        if (F32OUT) { dk32[e] = ak[c] * scale; dv32[e] = av[c]; }
        else { dk[e] = from_f<T>(ak[c] * scale); dv[e] = from_f<T>(av[c]); }
    }
}

// Partial dw / dbias over one (b, chunk of CHUNK positions) for head h: thread c owns channel c of x = [k ; v].
template <typename T>
__global__ void bwd_conv_partial_kernel(const T* __restrict__ k, const T* __restrict__ v, const float* __restrict__ dz,
                                        float* __restrict__ part_w, float* __restrict__ part_b, int B, int H, int Tlen,
                                        int D, int K, int nchunk)
{
    extern __shared__ float s_dz[];                 // CHUNK + K - 1 values: dz[j0-half .. j0+CHUNK-1+half]
    const int half = K / 2;
    const int h = blockIdx.y;
    const int b = blockIdx.x / nchunk, ch = blockIdx.x % nchunk;
    const int bh = b * H + h;
    const int p0 = ch * CHUNK;                      // rows p0 .. p0+CHUNK-1 of x
    // row p contributes to tap t through dz[p - t + half]
    for (int a = threadIdx.x; a < CHUNK + K - 1; a += blockDim.x) {
        const int j = p0 - half + a;
        s_dz[a] = (j >= 0 && j + half <= Tlen - 1) ? dz[(size_t)bh * Tlen + j] : 0.f;
    }
    __syncthreads();
    const int c = threadIdx.x;                      // 0 .. 2D-1
    float acc[kMaxTaps];
#pragma unroll
    for (int t = 0; t < kMaxTaps; ++t) acc[t] = 0.f;
    const T* src = c < D ? k : v;
    const int cc = c < D ? c : c - D;
    const int pend = p0 + CHUNK < Tlen ? p0 + CHUNK : Tlen;
#pragma unroll 8
    for (int p = p0; p < pend; ++p) {
        const float x = to_f(src[((size_t)bh * Tlen + p) * D + cc]);
#pragma unroll
        for (int t = 0; t < kMaxTaps; ++t)
            if (t < K) acc[t] = fmaf(s_dz[(p - p0) - t + 2 * half], x, acc[t]);   // dz index j = p - t + half
    }
    float* out = part_w + ((size_t)h * B * nchunk + blockIdx.x) * K * 2 * D;
#pragma unroll
    for (int t = 0; t < kMaxTaps; ++t)
        if (t < K) out[(size_t)t * 2 * D + c] = acc[t];
    if (threadIdx.x == 0) {
        // bias partial: the dz of the positions j in [p0, p0+CHUNK) themselves
        float sb = 0.f;
        for (int a = 0; a < CHUNK; ++a) sb += s_dz[a + half];
        part_b[(size_t)h * B * nchunk + blockIdx.x] = sb;
    }
}

__global__ void bwd_conv_reduce_kernel(const float* __restrict__ part_w, const float* __restrict__ part_b,
                                       float* __restrict__ dw, float* __restrict__ dbias, int nparts, int per_head)
{
    pdl_launch_dependents();
    pdl_wait();                                                // see launch_pdl: earlier kernels of the stream have completed
    const int h = blockIdx.y;
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e < per_head) {
        float s = 0.f;
        for (int p = 0; p < nparts; ++p) s += part_w[((size_t)h * nparts + p) * per_head + e];
        dw[(size_t)h * per_head + e] = s;
    }
    if (dbias && blockIdx.x == 0 && threadIdx.x == 0) {
        float s = 0.f;
        for (int p = 0; p < nparts; ++p) s += part_b[(size_t)h * nparts + p];
        dbias[h] = s;
    }
}

// dk, dv <- fp32 attention gradients + the scorer's input gradient, rounded once.
template <typename T>
__global__ void bwd_finish_kernel(const float* __restrict__ dk32, const float* __restrict__ dv32,
                                  const float* __restrict__ dz, const float* __restrict__ w, T* __restrict__ dk,
                                  T* __restrict__ dv, int H, int Tlen, int D, int K)
{
    const int half = K / 2;
    const size_t n = (size_t)gridDim.y * Tlen * D;
    const int bh = blockIdx.y;
    (void)n;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < Tlen * D; e += gridDim.x * blockDim.x) {
        const int p = e / D, c = e % D;
        const int h = bh % H;
        float gk = 0.f, gv = 0.f;
        for (int t = 0; t < K; ++t) {
            const int j = p - t + half;
            if (j < 0 || j + half > Tlen - 1) continue;
            const float g = dz[(size_t)bh * Tlen + j];
            gk = fmaf(g, w[((size_t)h * K + t) * 2 * D + c], gk);
            gv = fmaf(g, w[((size_t)h * K + t) * 2 * D + D + c], gv);
        }
        const size_t a = (size_t)bh * Tlen * D + e;
        dk[a] = from_f<T>(dk32[a] + gk);
        dv[a] = from_f<T>(dv32[a] + gv);
    }
}

// Tensor-core path: the scorer's input gradient sum_t dz[p-t+half] w[h,t,c] added in place onto the bf16 dk, dv rows.
// A block takes ROWS consecutive positions of one (b,h); 8 channels per thread, weights and the dz window in shared memory.
template <int D>
__global__ void __launch_bounds__(256) bwd_finish_inplace_kernel(const float* __restrict__ dz, const float* __restrict__ w,
                                                                 __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                                                                 int H, int Tlen, int K)
{
    constexpr int TPR = D / 8;                      // threads per row
    constexpr int RPP = 256 / TPR;                  // rows per pass
    constexpr int ROWS = 4 * RPP;
    extern __shared__ float sm[];
    float* ws = sm;                                 // [K][2D]
    float* dzs = sm + K * 2 * D;                    // dz[p0-half .. p0+ROWS-1+half]
    const int half = K / 2;
    const int bh = blockIdx.y, h = bh % H;
    const int p0 = blockIdx.x * ROWS;
    for (int i = threadIdx.x; i < K * 2 * D; i += 256) ws[i] = w[(size_t)h * K * 2 * D + i];
    for (int a = threadIdx.x; a < ROWS + K - 1; a += 256) {
        const int j = p0 - half + a;
        dzs[a] = (j >= 0 && j + half <= Tlen - 1) ? dz[(size_t)bh * Tlen + j] : 0.f;
    }
    __syncthreads();
    const int cc = (threadIdx.x % TPR) * 8, r0 = threadIdx.x / TPR;
#pragma unroll
    for (int ps = 0; ps < 4; ++ps) {
        const int rl = ps * RPP + r0, p = p0 + rl;
        if (p >= Tlen) break;
        float gk[8], gv[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) { gk[e] = 0.f; gv[e] = 0.f; }
        for (int t = 0; t < K; ++t) {
            const float g = dzs[rl - t + 2 * half];          // dz[p - t + half]
            const float4* wk = reinterpret_cast<const float4*>(&ws[(t * 2) * D + cc]);
            const float4* wv = reinterpret_cast<const float4*>(&ws[(t * 2 + 1) * D + cc]);
            const float4 a = wk[0], b = wk[1], c = wv[0], d = wv[1];
            gk[0] = fmaf(g, a.x, gk[0]); gk[1] = fmaf(g, a.y, gk[1]); gk[2] = fmaf(g, a.z, gk[2]); gk[3] = fmaf(g, a.w, gk[3]);
            gk[4] = fmaf(g, b.x, gk[4]); gk[5] = fmaf(g, b.y, gk[5]); gk[6] = fmaf(g, b.z, gk[6]); gk[7] = fmaf(g, b.w, gk[7]);
            gv[0] = fmaf(g, c.x, gv[0]); gv[1] = fmaf(g, c.y, gv[1]); gv[2] = fmaf(g, c.z, gv[2]); gv[3] = fmaf(g, c.w, gv[3]);
            gv[4] = fmaf(g, d.x, gv[4]); gv[5] = fmaf(g, d.y, gv[5]); gv[6] = fmaf(g, d.z, gv[6]); gv[7] = fmaf(g, d.w, gv[7]);
        }
        const size_t a0 = ((size_t)bh * Tlen + p) * D + cc;
        uint4 uk = *reinterpret_cast<const uint4*>(dk + a0), uv = *reinterpret_cast<const uint4*>(dv + a0);
        uint32_t kw[4] = {uk.x, uk.y, uk.z, uk.w}, vw[4] = {uv.x, uv.y, uv.z, uv.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 hk = __floats2bfloat162_rn(__uint_as_float(kw[e] << 16) + gk[2 * e],
                                                      __uint_as_float(kw[e] & 0xffff0000u) + gk[2 * e + 1]);
            __nv_bfloat162 hv = __floats2bfloat162_rn(__uint_as_float(vw[e] << 16) + gv[2 * e],
                                                      __uint_as_float(vw[e] & 0xffff0000u) + gv[2 * e + 1]);
            kw[e] = *reinterpret_cast<uint32_t*>(&hk);
            vw[e] = *reinterpret_cast<uint32_t*>(&hv);
        }
        *reinterpret_cast<uint4*>(dk + a0) = make_uint4(kw[0], kw[1], kw[2], kw[3]);
        *reinterpret_cast<uint4*>(dv + a0) = make_uint4(vw[0], vw[1], vw[2], vw[3]);
    }
}

// Tensor-core path, K = 5 or 7: one pass over the rows of k, v, dk, dv finishes the backward.  It first turns Eq. 6's inner
// products into logit gradients for the block's positions (and the taps around them): dr = the window share the dk/dv kernel
// wrote + the far-query share of a retained key (+ lambda where the token passes the threshold, Eq. 7), dz = dr r (1 - r);
// the retained keys' far-query shares of dk, dv (fp32, one row per list entry) are added onto their rows in the same
// pass, so that a retained row is rounded once.  Then both scorer jobs:  A block takes `rows`
// consecutive positions of one (b,h); a thread owns 4 channels of x = [k ; v] for every row it visits, so its
// K x 4 scorer weights stay in registers, and walks the block's rows: dw partials acc[t][c] += dz[p - t + half] x[p][c],
// and (FINISH) the scorer's input gradient sum_t dz[p - t + half] w[h,t,c] added onto the bf16 dk, dv rows in place.
// The partials of the threads that own the same channels are added in a fixed order (a tree over the row slots
// through shared memory).
__device__ __forceinline__ bool isv_of(int cg, int D) { return cg >= D / 4; }
constexpr int TAIL_MIN_ROWS = 256, TAIL_MAX_ROWS = 1024;   // rows per block are chosen per launch to fill whole waves
template <int D, int K, bool FINISH>
__global__ void __launch_bounds__(256, 2)
bwd_tail_kernel(const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, const float* __restrict__ dr_win,
                const float* __restrict__ z, const float* __restrict__ lambda, const int32_t* __restrict__ idx,
                const int32_t* __restrict__ cnt, const float* __restrict__ dk_ret, const float* __restrict__ dv_ret,
                const float* __restrict__ dr_ret, const float* __restrict__ w, __nv_bfloat16* __restrict__ dk,
                __nv_bfloat16* __restrict__ dv, float* __restrict__ part_w, float* __restrict__ part_b, int B, int H, int Tlen,
                int R, float zthr, int nchunk, int rows)
{
    pdl_launch_dependents();
    pdl_wait();                                                // see launch_pdl: earlier kernels of the stream have completed
    constexpr int TPR = 2 * D / 4;                  // threads per position: D/4 for k, D/4 for v
    constexpr int RPP = 256 / TPR;                  // positions per pass (row slots)
    constexpr int half = K / 2;
    const int NDZ = (rows + K - 1 + 3) & ~3;
    extern __shared__ float sm[];
    float* dzs = sm;                                // dz[p0-half .. p0+rows-1+half]
    int* ent = reinterpret_cast<int*>(dzs + NDZ);   // list entry of the same positions, or -1
    float* red = dzs + 2 * NDZ;                     // [RPP/2][K][2D]
    const int h = blockIdx.y;
    const int b = blockIdx.x / nchunk, ch = blockIdx.x % nchunk;
    const int bh = b * H + h;
    const int p0 = ch * rows;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int a = tid; a < rows + K - 1; a += 256) ent[a] = -1;
    __syncthreads();
    {
        const int n_ret = cnt[bh];
        const int32_t* id = idx + (size_t)bh * R;
        for (int e = tid; e < n_ret; e += 256) {
            const int a = id[e] - (p0 - half);
            if (a >= 0 && a < rows + K - 1) ent[a] = e;
        }
    }
    __syncthreads();
    for (int a = tid; a < rows + K - 1; a += 256) {
        const int j = p0 - half + a;
        float g = 0.f;
        if (j >= 0 && j + half <= Tlen - 1) {       // scored tokens only
            float dr = dr_win[(size_t)bh * Tlen + j];
            if (ent[a] >= 0) dr += dr_ret[(size_t)bh * R + ent[a]];
            const float zz = z[(size_t)bh * Tlen + j];
            const float r = 1.f / (1.f + expf(-zz));
            if (lambda && zz > zthr) dr += lambda[h];
            g = dr * r * (1.f - r);
        }
        dzs[a] = g;
    }
    const int cg = tid % TPR, r0 = tid / TPR;       // channel group: x channels [4 cg, 4 cg + 4); row slot
    const float* gret = isv_of(cg, D) ? dv_ret : dk_ret;
    const bool isv = cg >= D / 4;
    const int cc = (cg % (D / 4)) * 4;              // first of this thread's 4 channels within k or v
    const __nv_bfloat16* src = isv ? v : k;
    __nv_bfloat16* gdst = isv ? dv : dk;
    // the multiply-adds run on packed fp32 pairs (channels 0,1 and 2,3 of the thread's four): the loop is bound by
    // instruction issue, not by memory
    using tc::pack2; using tc::unpack2; using tc::fma2;
    uint64_t wr2[K][2];                             // this thread's scorer weights
    if (FINISH) {
#pragma unroll
        for (int t = 0; t < K; ++t) {
            const float4 w4 = *reinterpret_cast<const float4*>(&w[((size_t)h * K + t) * 2 * D + cg * 4]);
            wr2[t][0] = pack2(w4.x, w4.y); wr2[t][1] = pack2(w4.z, w4.w);
        }
    }
    __syncthreads();
    uint64_t acc2[K][2];
#pragma unroll
    for (int t = 0; t < K; ++t) acc2[t][0] = acc2[t][1] = pack2(0.f, 0.f);
    // U rows per batch: all of a batch's loads are issued before any of its arithmetic (row indices are clamped so
    // that every load is legal; rows past the end are skipped afterwards)
    constexpr int U = 8;
    for (int rb = r0; rb < rows; rb += RPP * U) {
        uint2 ux[U], ug[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int p = min(p0 + rb + u * RPP, Tlen - 1);
            const size_t a0 = ((size_t)bh * Tlen + p) * D + cc;
            ux[u] = *reinterpret_cast<const uint2*>(src + a0);
            ug[u] = make_uint2(0u, 0u);
            if (FINISH || ent[min(rb + u * RPP, rows - 1) + half] >= 0) ug[u] = *reinterpret_cast<const uint2*>(gdst + a0);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int rl = rb + u * RPP, p = p0 + rl;
            if (rl >= rows || p >= Tlen) continue;
            uint64_t g2[K];
            const uint64_t x01 = pack2(__uint_as_float(ux[u].x << 16), __uint_as_float(ux[u].x & 0xffff0000u));
            const uint64_t x23 = pack2(__uint_as_float(ux[u].y << 16), __uint_as_float(ux[u].y & 0xffff0000u));
#pragma unroll
            for (int t = 0; t < K; ++t) { const float g = dzs[rl - t + 2 * half]; g2[t] = pack2(g, g); }   // dz[p - t + half]
#pragma unroll
            for (int t = 0; t < K; ++t) { acc2[t][0] = fma2(g2[t], x01, acc2[t][0]); acc2[t][1] = fma2(g2[t], x23, acc2[t][1]); }
            const int er = ent[rl + half];                   // retained: its far-query share is added here
            if (FINISH || er >= 0) {
                float gi[4] = {0.f, 0.f, 0.f, 0.f};
                if (FINISH) {
                    uint64_t gi01 = pack2(0.f, 0.f), gi23 = gi01;
#pragma unroll
                    for (int t = 0; t < K; ++t) { gi01 = fma2(g2[t], wr2[t][0], gi01); gi23 = fma2(g2[t], wr2[t][1], gi23); }
                    unpack2(gi01, gi[0], gi[1]); unpack2(gi23, gi[2], gi[3]);
                }
                if (er >= 0) {
                    const float4 f4 = *reinterpret_cast<const float4*>(gret + ((size_t)bh * R + er) * D + cc);
                    gi[0] += f4.x; gi[1] += f4.y; gi[2] += f4.z; gi[3] += f4.w;
                }
                __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(ug[u].x << 16) + gi[0], __uint_as_float(ug[u].x & 0xffff0000u) + gi[1]);
                __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(ug[u].y << 16) + gi[2], __uint_as_float(ug[u].y & 0xffff0000u) + gi[3]);
                *reinterpret_cast<uint2*>(gdst + ((size_t)bh * Tlen + p) * D + cc) =
                    make_uint2(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1));
            }
        }
    }
    float acc[K][4];
#pragma unroll
    for (int t = 0; t < K; ++t) { unpack2(acc2[t][0], acc[t][0], acc[t][1]); unpack2(acc2[t][1], acc[t][2], acc[t][3]); }
    // ---- add the partials of the row slots: slots [step, 2 step) hand their sums to slots [0, step) ---------
#pragma unroll
    for (int step = RPP / 2; step >= 1; step >>= 1) {
        if (r0 >= step && r0 < 2 * step) {
            float* dst = red + (size_t)(r0 - step) * K * 2 * D;
#pragma unroll
            for (int t = 0; t < K; ++t)
                *reinterpret_cast<float4*>(&dst[t * 2 * D + cg * 4]) = make_float4(acc[t][0], acc[t][1], acc[t][2], acc[t][3]);
        }
        __syncthreads();
        if (r0 < step) {
            const float* s2 = red + (size_t)r0 * K * 2 * D;
#pragma unroll
            for (int t = 0; t < K; ++t) {
                const float4 a = *reinterpret_cast<const float4*>(&s2[t * 2 * D + cg * 4]);
                acc[t][0] += a.x; acc[t][1] += a.y; acc[t][2] += a.z; acc[t][3] += a.w;
            }
        }
        __syncthreads();
    }
    if (r0 == 0) {
        float* out = part_w + ((size_t)h * B * nchunk + blockIdx.x) * K * 2 * D;
#pragma unroll
        for (int t = 0; t < K; ++t)
            *reinterpret_cast<float4*>(&out[t * 2 * D + cg * 4]) = make_float4(acc[t][0], acc[t][1], acc[t][2], acc[t][3]);
    }
    if (warp == 7) {                                // bias partial: the dz of the block's own positions
        float sb = 0.f;
        for (int a = lane; a < rows; a += 32) sb += dzs[a + half];
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) sb += __shfl_xor_sync(0xffffffffu, sb, o);
        if (lane == 0) part_b[(size_t)h * B * nchunk + blockIdx.x] = sb;
    }
}

// Rows per block for the fused pass: between TAIL_MIN_ROWS and TAIL_MAX_ROWS, such that the grid fills whole waves of
// the resident-block slots as well as possible (ties: fewer, larger blocks).  Returns the chunks per sequence.
inline int tail_chunks(const Params& p, int* rows_out)
{
    int sms = 148;
    device_sm_count(&sms);
    const int slots = 2 * sms;
    const int lo = (p.T + TAIL_MAX_ROWS - 1) / TAIL_MAX_ROWS, hi = (p.T + TAIL_MIN_ROWS - 1) / TAIL_MIN_ROWS;
    int best = lo;
    double best_eff = -1.0;
    for (int n = lo; n <= hi; ++n) {
        const double waves = (double)p.B * p.H * n / slots;
        const double eff = waves / (double)(long long)(waves + 0.999999);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = n; }
    }
    int rows = (p.T + best - 1) / best;
    rows = (rows + 7) / 8 * 8;                      // a multiple of every kernel's rows per pass
    *rows_out = rows;
    return (p.T + rows - 1) / rows;
}

template <int D, int K>
int run_tail(const Params& p, const void* k, const void* v, const float* dr_win, const float* z, const float* lambda,
             const int32_t* idx, const int32_t* cnt, const float* ret_ws, void* dk, void* dv, float* part_w, float* part_b,
             bool finish, int nchunk, int rows, cudaStream_t st)
{
    const size_t sm = (size_t)(2 * ((rows + K - 1 + 3) & ~3) + (256 / (2 * D / 4) / 2) * K * 2 * D) * sizeof(float);
    dim3 grid(p.B * nchunk, p.H);
    // the retained tiles' scratch: dk_ret, dv_ret [B,H,R,d], dr_ret [B,H,R] (layout of launch_bwd_dkv_tc)
    const size_t n = (size_t)p.B * p.H * (p.R > 0 ? p.R : 1);
    const float* dk_ret = ret_ws; const float* dv_ret = dk_ret + n * D; const float* dr_ret = dv_ret + n * D;
    if (finish)
        launch_pdl(bwd_tail_kernel<D, K, true>, grid, dim3(256), sm, st, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, dr_win, z,
                   lambda, idx, cnt, dk_ret, dv_ret, dr_ret, p.w, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, part_w, part_b, p.B, p.H,
                   p.T, p.R, p.zthr, nchunk, rows);
    else
        launch_pdl(bwd_tail_kernel<D, K, false>, grid, dim3(256), sm, st, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, dr_win, z,
                   lambda, idx, cnt, dk_ret, dv_ret, dr_ret, p.w, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, part_w, part_b, p.B, p.H,
                   p.T, p.R, p.zthr, nchunk, rows);
    return cuda_status(cudaGetLastError());
}

struct WsPlan { size_t delta, dz, part_w, part_b, dk32, dv32, ret, total; int nchunk; };
WsPlan plan(const Params& p, uint32_t flags)
{
    WsPlan w;
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    const size_t bht = (size_t)p.B * p.H * p.T;
    w.nchunk = (p.T + CHUNK - 1) / CHUNK;
    size_t off = 0;
    w.delta = off; off += up(bht * p.G * 4);        // one per query head
    w.dz = off; off += up(bht * 4);
    if (p.stack) {                                  // the stack's backward keeps one packed partial gradient per CTA
        const size_t a = stack_bwd_workspace(p), b = stack_bwd_tc_workspace(p);
        w.part_w = off; off += up(a > b ? a : b);
        w.part_b = off;
    } else {
        w.part_w = off; off += up((size_t)p.H * p.B * w.nchunk * p.K * 2 * p.d * 4);
        w.part_b = off; off += up((size_t)p.H * p.B * w.nchunk * 4);
    }
    w.dk32 = w.dv32 = 0;
    const bool tc_path = p.dtype == LTE_BF16 && (p.d == 32 || p.d == 64 || p.d == 128);
    if ((flags & LTE_BWD_CNN_INPUT_GRAD) && !tc_path && !p.stack) {
        w.dk32 = off; off += up(bht * p.d * 4);
        w.dv32 = off; off += up(bht * p.d * 4);
    }
    w.ret = off;
    if (tc_path) off += bwd_tc_ret_bytes(p);        // tensor-core path: retained-tile shares
    w.total = off;
    return w;
}

template <typename T, int D>
int run(const Params& p, const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dO,
        const float* z, const int32_t* idx, const int32_t* cnt, const float* lambda, void* dq, void* dk, void* dv,
        float* dw, float* dbias, uint32_t flags, void* ws, cudaStream_t st)
{
    const WsPlan w = plan(p, flags);
    char* base = (char*)ws;
    float* delta = (float*)(base + w.delta);
    float* dz = (float*)(base + w.dz);
    float* part_w = (float*)(base + w.part_w);
    float* part_b = (float*)(base + w.part_b);
    float* dk32 = (float*)(base + w.dk32);
    float* dv32 = (float*)(base + w.dv32);
    const bool want_in = flags & LTE_BWD_CNN_INPUT_GRAD;
    const bool f32 = want_in && !p.stack;             // the stack's backward adds its input gradient to dk, dv in place
    dim3 grid((p.T + 3) / 4, p.B * p.H), gridq((p.T + 3) / 4, p.B * p.H * p.G);
    if constexpr (sizeof(T) == 2 && (D == 32 || D == 64 || D == 128)) {
        const int e = launch_bwd_dq_tc(p, q, k, v, o, lse, dO, idx, cnt, dq, delta, st);
        if (e != LTE_OK) return e;
    } else {
        bwd_dq_kernel<T, D><<<gridq, 128, 0, st>>>((const T*)q, (const T*)k, (const T*)v, (const T*)o, (const T*)dO, lse,
                                                   idx, cnt, (T*)dq, delta, p.T, p.W, p.R, p.scale, p.G);
    }
    if constexpr (sizeof(T) == 2 && (D == 32 || D == 64 || D == 128)) {
        // K = 5 or 7 with the single layer: the last pass (bwd_tail_kernel) also merges the retained shares and forms dz
        const bool tail_merges = !p.stack && (p.K == 5 || p.K == 7);
        const int e = launch_bwd_dkv_tc(p, q, k, v, lse, dO, delta, z, idx, cnt, lambda, dk, dv, dk32, dv32, dz, base + w.ret,
                                        false, !tail_merges, st);
        if (e != LTE_OK) return e;
    } else if (f32) {
        bwd_dkv_kernel<T, D, true><<<grid, 128, 0, st>>>((const T*)q, (const T*)k, (const T*)v, (const T*)dO, lse, delta,
                                                         z, idx, cnt, lambda, (T*)dk, (T*)dv, dk32, dv32, dz, p.H, p.T,
                                                         p.W, p.R, p.half, p.zthr, p.scale, p.G);
    } else {
        bwd_dkv_kernel<T, D, false><<<grid, 128, 0, st>>>((const T*)q, (const T*)k, (const T*)v, (const T*)dO, lse, delta,
                                                          z, idx, cnt, lambda, (T*)dk, (T*)dv, dk32, dv32, dz, p.H, p.T,
                                                          p.W, p.R, p.half, p.zthr, p.scale, p.G);
    }
    if (p.stack) {                                  // bf16: tensor cores; fp32 storage: the fp32 kernel
        if (stack_bwd_tc_workspace(p) > 0) return launch_stack_bwd_tc(p, k, v, dz, dk, dv, dw, dbias, want_in, part_w, st);
        return launch_stack_bwd(p, k, v, dz, dk, dv, dw, dbias, want_in, part_w, st);
    }
    const int per_head = p.K * 2 * D;
    dim3 gr((per_head + 255) / 256, p.H);
    if constexpr (sizeof(T) == 2 && (D == 32 || D == 64 || D == 128)) {
        if (p.K == 5 || p.K == 7) {                   // fused pass: dw partials and the scorer's input gradient
            int rows = 0;
            const int nch = tail_chunks(p, &rows);
            const float* rw = (const float*)(base + w.ret);
            const int e = p.K == 7 ? run_tail<D, 7>(p, k, v, dz, z, lambda, idx, cnt, rw, dk, dv, part_w, part_b, f32, nch, rows, st)
                                   : run_tail<D, 5>(p, k, v, dz, z, lambda, idx, cnt, rw, dk, dv, part_w, part_b, f32, nch, rows, st);
            if (e != LTE_OK) return e;
            launch_pdl(bwd_conv_reduce_kernel, gr, dim3(256), 0, st, part_w, part_b, dw, dbias, p.B * nch, per_head);
            return cuda_status(cudaGetLastError());
        }
    }
    dim3 gc(p.B * w.nchunk, p.H);
    bwd_conv_partial_kernel<T><<<gc, 2 * D, (CHUNK + p.K - 1) * sizeof(float), st>>>(
        (const T*)k, (const T*)v, dz, part_w, part_b, p.B, p.H, p.T, D, p.K, w.nchunk);
    bwd_conv_reduce_kernel<<<gr, 256, 0, st>>>(part_w, part_b, dw, dbias, p.B * w.nchunk, per_head);
    if (f32) {
        if constexpr (sizeof(T) == 2 && (D == 32 || D == 64 || D == 128)) {
            constexpr int ROWS = 4 * (256 / (D / 8));
            dim3 gf((p.T + ROWS - 1) / ROWS, p.B * p.H);
            const size_t sm = (size_t)(p.K * 2 * D + ROWS + p.K - 1) * sizeof(float);
            bwd_finish_inplace_kernel<D><<<gf, 256, sm, st>>>(dz, p.w, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, p.H, p.T, p.K);
        } else {
            dim3 gf(min((p.T * D + 255) / 256, 1024), p.B * p.H);
            bwd_finish_kernel<T><<<gf, 256, 0, st>>>(dk32, dv32, dz, p.w, (T*)dk, (T*)dv, p.H, p.T, D, p.K);
        }
    }
    return cuda_status(cudaGetLastError());
}

}  // namespace

size_t bwd_workspace_bytes(const Params& p, uint32_t flags) { return plan(p, flags).total; }

int launch_bwd(const Params& p, const void* q, const void* k, const void* v, const void* o, const float* lse,
               const void* dO, const float* z, const int32_t* idx, const int32_t* cnt, const float* lambda, void* dq,
               void* dk, void* dv, float* dw, float* dbias, uint32_t flags, void* ws, cudaStream_t st)
{
#define LTE_GO(T, D) \
    return run<T, D>(p, q, k, v, o, lse, dO, z, idx, cnt, lambda, dq, dk, dv, dw, dbias, flags, ws, st)
    if (p.dtype == LTE_BF16) {
        switch (p.d) { case 32: LTE_GO(__nv_bfloat16, 32); case 64: LTE_GO(__nv_bfloat16, 64); case 128: LTE_GO(__nv_bfloat16, 128); }
    } else {
        switch (p.d) { case 32: LTE_GO(float, 32); case 64: LTE_GO(float, 64); case 128: LTE_GO(float, 128); }
    }
#undef LTE_GO
    return LTE_ERR_UNSUPPORTED;
}

}  // namespace lte
