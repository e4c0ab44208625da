// Prefill attention on the plain fp32 ALUs: the fp32 storage path (every product and sum in fp32).
// One warp per query; the d channels are spread over the lanes, keys are visited one by one
// (retained entries already out of the query's window first, then the window), online softmax.
// This is the reference-precision path for fp32 tensors; bf16 tensors use the tensor-core kernel.
// With `leave` (the streaming reading of a chunked prefill) list entry a is visible to query i only while i < leave[a]:
// the entry was pushed out of the pool by a better token at that query.
#include "common.cuh"

namespace lte {
namespace {

template <typename T, int D>
__global__ void __launch_bounds__(128) prefill_simt_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                           const T* __restrict__ v, const int32_t* __restrict__ idx,
                                                           const int32_t* __restrict__ cnt, T* __restrict__ o,
                                                           float* __restrict__ lse, int Tlen, int W, int R, float scale, int G, int qoff,
                                                           const int32_t* __restrict__ leave)
{
    constexpr int C = D / 32;                  // channels per lane
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = qoff + blockIdx.x * 4 + warp;     // position; q, o, lse hold the queries from position qoff on
    const int bh = blockIdx.y, bhk = bh / G;   // query head and its key/value head
    if (i >= Tlen) return;
    const size_t base = ((size_t)bh * (Tlen - qoff) + (i - qoff)) * D, kbase = (size_t)bhk * Tlen * D;   // this query's row of q and o
    float qv[C], acc[C];
#pragma unroll
    for (int c = 0; c < C; ++c) { qv[c] = to_f(q[base + lane + 32 * c]) * scale; acc[c] = 0.f; }
    float m = -INFINITY, l = 0.f;
    const int32_t* id = idx + (size_t)bhk * R;
    const int32_t* lv = leave ? leave + (size_t)bhk * R : nullptr;
    const int n_ret = cnt[bhk];
    const int lo = i - W + 1 > 0 ? i - W + 1 : 0;
    // number of retained entries visible to this query: idx ascending => a prefix
    int nvis = 0;
    for (int m0 = 0; m0 < n_ret; m0 += 32) {
        int e = m0 + lane < n_ret ? id[m0 + lane] : 0x7fffffff;
        unsigned b = __ballot_sync(0xffffffffu, e <= i - W);
        nvis += __popc(b);
        if (b != 0xffffffffu) break;
    }
    const int total = nvis + (i - lo + 1);
    for (int a = 0; a < total; ++a) {
        if (lv && a < nvis && lv[a] <= i) continue;                 // no longer in the pool at this query
        const int j = a < nvis ? id[a] : lo + (a - nvis);
        const T* kr = k + kbase + (size_t)j * D;
        const T* vr = v + kbase + (size_t)j * D;
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < C; ++c) s = fmaf(qv[c], to_f(kr[lane + 32 * c]), s);
        s = warp_sum(s);
        const float mn = fmaxf(m, s);
        const float alpha = expf(m - mn), pj = expf(s - mn);
        l = l * alpha + pj;
#pragma unroll
        for (int c = 0; c < C; ++c) acc[c] = fmaf(pj, to_f(vr[lane + 32 * c]), acc[c] * alpha);
        m = mn;
    }
    const float inv = 1.f / l;
#pragma unroll
    for (int c = 0; c < C; ++c) o[base + lane + 32 * c] = from_f<T>(acc[c] * inv);
    if (lane == 0) lse[(size_t)bh * (Tlen - qoff) + (i - qoff)] = m + logf(l);
}

template <typename T>
int run(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx, const int32_t* cnt,
        void* o, float* lse, const int32_t* leave, cudaStream_t st)
{
    dim3 grid((p.T - p.qoff + 3) / 4, p.B * p.H * p.G);
#define LTE_GO(D)                                                                                          \
    prefill_simt_kernel<T, D><<<grid, 128, 0, st>>>((const T*)q, (const T*)k, (const T*)v, idx, cnt, (T*)o, \
                                                    lse, p.T, p.W, p.R, p.scale, p.G, p.qoff, leave)
    switch (p.d) {
        case 32: LTE_GO(32); break;
        case 64: LTE_GO(64); break;
        case 128: LTE_GO(128); break;
        default: return LTE_ERR_UNSUPPORTED;
    }
#undef LTE_GO
    return cuda_status(cudaGetLastError());
}

}  // namespace

int launch_prefill_simt(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx,
                        const int32_t* cnt, void* o, float* lse, cudaStream_t st, const int32_t* leave)
{
    return p.dtype == LTE_BF16 ? run<__nv_bfloat16>(p, q, k, v, idx, cnt, o, lse, leave, st)
                               : run<float>(p, q, k, v, idx, cnt, o, lse, leave, st);
}

}  // namespace lte
