// Retention logits of the single-layer scorer (Section 3.1.1): z_j = bias + sum_t <w_t, x_{j+t-half}>.
//
// Each input row x_p = [k_p ; v_p] is read from HBM once per tile and turned into K partial dot
// products Y[p][t] = <w_t, x_p> by one thread (weights broadcast from shared memory, fp32 FMA);
// the logit of token j is then the shifted diagonal sum_t Y[j+t-half][t], taken from shared memory.
// A block of NT threads covers NT rows and emits NT-(K-1) logits; the K-1 halo rows are recomputed by
// the neighbouring block.  HBM traffic: 2*d elements read and one fp32 written per token and head.
#include "common.cuh"

namespace lte {
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

template <typename T, int D, int K>
int run(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    constexpr int TJ = NT - (K - 1);
    dim3 grid((p.T + TJ - 1) / TJ, p.B * p.H);
    scores_kernel<T, D, K><<<grid, NT, 0, st>>>((const T*)k, (const T*)v, p.w, p.bias, z, r, p.H, p.T);
    return cuda_status(cudaGetLastError());
}

template <typename T, int D>
int by_k(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    switch (p.K) {
        case 1: return run<T, D, 1>(p, k, v, z, r, st);
        case 3: return run<T, D, 3>(p, k, v, z, r, st);
        case 5: return run<T, D, 5>(p, k, v, z, r, st);
        case 7: return run<T, D, 7>(p, k, v, z, r, st);
        case 9: return run<T, D, 9>(p, k, v, z, r, st);
        case 11: return run<T, D, 11>(p, k, v, z, r, st);
        case 13: return run<T, D, 13>(p, k, v, z, r, st);
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

int launch_scores(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    return p.dtype == LTE_BF16 ? by_d<__nv_bfloat16>(p, k, v, z, r, st) : by_d<float>(p, k, v, z, r, st);
}

}  // namespace lte
