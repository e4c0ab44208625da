// The training-free selection rules the paper's ablation compares with (Section 4, last paragraph), behind the same
// retained-list interface as the learned rule:
//   uniform stride + window   out-of-window tokens kept at a uniform stride (the sink first): no scores involved
//   accumulated attention     every out-of-window token is a candidate and the R with the largest accumulated attention
//                             a_j = sum_i P_ij stay: the ranking is lte_select's without a threshold; this file computes a_j
// Neither is on the hot path of the learned rule: plain kernels.
#include "common.cuh"

namespace lte {
namespace {

// One thread block per (b,h): positions 0 .. min(sink, E, R) - 1, then sink, sink + stride, ... < E with the smallest
// stride that fits the remaining slots.  E = max(T - W, 0).
__global__ void select_uniform_kernel(int32_t* __restrict__ idx, int32_t* __restrict__ cnt, int32_t* __restrict__ ncand,
                                      int Tlen, int W, int R, int sink)
{
    const int bh = blockIdx.x;
    const int E = Tlen - W > 0 ? Tlen - W : 0;
    const int ns = min(min(sink, E), R);
    const int n = R - ns, rest = E - min(sink, E);
    int stride = 1, nk = 0;
    if (n > 0 && rest > 0) { stride = (rest + n - 1) / n; if (stride < 1) stride = 1; nk = (rest + stride - 1) / stride; }
    for (int e = threadIdx.x; e < R; e += blockDim.x) {
        int v = -1;
        if (e < ns) v = e;
        else if (e - ns < nk) v = sink + (e - ns) * stride;
        idx[(size_t)bh * R + e] = v;
    }
    if (threadIdx.x == 0) { cnt[bh] = ns + nk; if (ncand) ncand[bh] = E; }
}

// Accumulated attention: one warp per key j of key/value head bh; over the queries that see j (the W window queries
// j .. j+W-1 and, if j is in the list, every query from j+W on) of every query head of the group:
// a_j = sum_i exp(scale q_i.k_j - lse_i).  Fixed summation order (deterministic).
template <typename T, int D>
__global__ void __launch_bounds__(128) colsum_kernel(const T* __restrict__ q, const T* __restrict__ k, const float* __restrict__ lse,
                                                     const int32_t* __restrict__ idx, const int32_t* __restrict__ cnt,
                                                     float* __restrict__ a, int Tlen, int W, int R, float scale, int G)
{
    constexpr int C = D / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = blockIdx.x * 4 + warp;
    const int bh = blockIdx.y;
    if (j >= Tlen) return;
    float kv[C];
#pragma unroll
    for (int c = 0; c < C; ++c) kv[c] = to_f(k[((size_t)bh * Tlen + j) * D + lane + 32 * c]) * scale;
    bool kept = false;
    {
        const int32_t* id = idx + (size_t)bh * R;
        int lo = 0, hi = cnt[bh];
        while (lo < hi) { const int mid = (lo + hi) >> 1; if (id[mid] < j) lo = mid + 1; else hi = mid; }
        kept = lo < cnt[bh] && id[lo] == j;
    }
    const int iend = kept ? Tlen - 1 : min(j + W - 1, Tlen - 1);
    float acc = 0.f;
    for (int g = 0; g < G; ++g) {
        const size_t qbase = ((size_t)bh * G + g) * Tlen;
        for (int i = j; i <= iend; ++i) {
            const T* qr = q + (qbase + i) * D;
            float s = 0.f;
#pragma unroll
            for (int c = 0; c < C; ++c) s = fmaf(to_f(qr[lane + 32 * c]), kv[c], s);
            s = warp_sum(s);
            acc += expf(s - lse[qbase + i]);
        }
    }
    if (lane == 0) a[(size_t)bh * Tlen + j] = acc;
}

}  // namespace

int launch_select_uniform(const Params& p, int32_t* idx, int32_t* cnt, int32_t* ncand, cudaStream_t st)
{
    select_uniform_kernel<<<p.B * p.H, 128, 0, st>>>(idx, cnt, ncand, p.T, p.W, p.R, p.sink);
    return cuda_status(cudaGetLastError());
}

int launch_colsum(const Params& p, const void* q, const void* k, const float* lse, const int32_t* idx, const int32_t* cnt,
                  float* a, cudaStream_t st)
{
    dim3 grid((p.T + 3) / 4, p.B * p.H);
#define LTE_GO(TY, D) colsum_kernel<TY, D><<<grid, 128, 0, st>>>((const TY*)q, (const TY*)k, lse, idx, cnt, a, p.T, p.W, p.R, p.scale, p.G)
    if (p.dtype == LTE_BF16) {
        switch (p.d) { case 32: LTE_GO(__nv_bfloat16, 32); break; case 64: LTE_GO(__nv_bfloat16, 64); break; case 128: LTE_GO(__nv_bfloat16, 128); break; default: return LTE_ERR_UNSUPPORTED; }
    } else {
        switch (p.d) { case 32: LTE_GO(float, 32); break; case 64: LTE_GO(float, 64); break; case 128: LTE_GO(float, 128); break; default: return LTE_ERR_UNSUPPORTED; }
    }
#undef LTE_GO
    return cuda_status(cudaGetLastError());
}

}  // namespace lte
