// Retention logits of the single-layer scorer (Section 3.1.1): z_j = bias + sum_t <w_t, x_{j+t-half}>.
//
// Each input row x_p = [k_p ; v_p] is read from HBM once per tile and turned into K partial dot
// products Y[p][t] = <w_t, x_p> by one thread (weights broadcast from shared memory, fp32 FMA);
// the logit of token j is then the shifted diagonal sum_t Y[j+t-half][t], taken from shared memory.
// A block of NT threads covers NT rows and emits NT-(K-1) logits; the K-1 halo rows are recomputed by
// the neighbouring block.  HBM traffic: 2*d elements read and one fp32 written per token and head.
#include "tma_util.cuh"

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

// ---- bf16, d = 64 or 128: the tile of input rows is staged by TMA -----------------------------------------------
// A block takes NT consecutive input rows of one (b,h): one cp.async.bulk.tensor box per 64-column sub-tile of k and
// of v (128-byte swizzle, so that thread r reading row r is bank-conflict free), rows left of position 0 or right of
// T-1 arriving as zeros, which is exactly the scorer's zero padding.  HBM is read by the copy engine only; the
// threads spend their issue slots on the K partial dot products per row (weights broadcast from shared memory).
__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

template <int D, int K>
__global__ void __launch_bounds__(NT) scores_tma_kernel(const __grid_constant__ CUtensorMap tmK,
                                                        const __grid_constant__ CUtensorMap tmV,
                                                        const float* __restrict__ w, const float* __restrict__ bias,
                                                        float* __restrict__ z, float* __restrict__ r, int H, int Tlen,
                                                        int* __restrict__ status)
{
    constexpr int HALF = K / 2;
    constexpr int TJ = NT - (K - 1);
    constexpr int SUB = D / 64;
    extern __shared__ __align__(1024) uint8_t smem[];
    // [k tile: SUB x 16 KB][v tile: SUB x 16 KB][weights K*2D floats][ys NT*K floats][mbarrier]
    float* ws = reinterpret_cast<float*>(smem + 2 * SUB * 16384);
    float* ys = ws + K * 2 * D;
    const uint32_t bar = s_u32(ys + NT * K);
    const uint32_t tile = s_u32(smem);
    const int bh = blockIdx.y, h = bh % H;
    const int j0 = blockIdx.x * TJ;
    const int tid = threadIdx.x;

    if ((tile & 1023u) != 0) { if (tid == 0) atomicExch(status, 8); return; }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(2 * SUB * 16384) : "memory");
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb) {
            asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                         ::"r"(tile + sb * 16384), "l"(&tmK), "r"(sb * 64), "r"(j0 - HALF), "r"(bh), "r"(bar) : "memory");
            asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                         ::"r"(tile + (SUB + sb) * 16384), "l"(&tmV), "r"(sb * 64), "r"(j0 - HALF), "r"(bh), "r"(bar) : "memory");
        }
    }
    for (int i = tid; i < K * 2 * D; i += NT) ws[i] = w[(size_t)h * K * 2 * D + i];
    __syncthreads();
    if (tid == 0) {                                     // one thread polls (bounded), the block barrier releases the rest
        uint32_t ok = 0;
        for (uint32_t it = 0; it < (1u << 22) && !ok; ++it)
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(bar) : "memory");
        if (!ok) atomicExch(status, 7);
    }
    __syncthreads();

    float acc[K];
#pragma unroll
    for (int t = 0; t < K; ++t) acc[t] = 0.f;
#pragma unroll
    for (int part = 0; part < 2; ++part) {
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb) {
            const uint8_t* rowp = smem + (part * SUB + sb) * 16384 + tid * 128;
#pragma unroll 2
            for (int ch = 0; ch < 8; ++ch) {
                const uint4 u = *reinterpret_cast<const uint4*>(rowp + ((ch ^ (tid & 7)) << 4));
                const uint32_t wd[4] = {u.x, u.y, u.z, u.w};
                float x[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) { x[2 * i] = __uint_as_float(wd[i] << 16); x[2 * i + 1] = __uint_as_float(wd[i] & 0xffff0000u); }
                const int c = sb * 64 + ch * 8;
#pragma unroll
                for (int t = 0; t < K; ++t) {
                    const float4* wv = reinterpret_cast<const float4*>(&ws[(t * 2 + part) * D + c]);
                    const float4 a = wv[0], b = wv[1];
                    acc[t] = fmaf(x[0], a.x, acc[t]); acc[t] = fmaf(x[1], a.y, acc[t]);
                    acc[t] = fmaf(x[2], a.z, acc[t]); acc[t] = fmaf(x[3], a.w, acc[t]);
                    acc[t] = fmaf(x[4], b.x, acc[t]); acc[t] = fmaf(x[5], b.y, acc[t]);
                    acc[t] = fmaf(x[6], b.z, acc[t]); acc[t] = fmaf(x[7], b.w, acc[t]);
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
            zz = -INFINITY;
        } else {
            zz = bias ? bias[h] : 0.f;
#pragma unroll
            for (int t = 0; t < K; ++t) zz += ys[(tid + t) * K + t];
        }
        z[(size_t)bh * Tlen + j] = zz;
        if (r) r[(size_t)bh * Tlen + j] = 1.f / (1.f + __expf(-zz));
    }
}

__device__ int g_scores_status = 0;

template <int D, int K>
int run_tma(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    constexpr int TJ = NT - (K - 1);
    constexpr int SMEM = 2 * (D / 64) * 16384 + (K * 2 * D + NT * K) * 4 + 16;
    CUtensorMap tk, tv;
    if (!make_map(&tk, k, p.B * p.H, p.T, D, NT) || !make_map(&tv, v, p.B * p.H, p.T, D, NT)) return LTE_ERR_CUDA;
    static bool attr_done = false;
    static int* status_ptr = nullptr;
    if (!attr_done) {
        if (cudaFuncSetAttribute(scores_tma_kernel<D, K>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess ||
            cudaGetSymbolAddress((void**)&status_ptr, g_scores_status) != cudaSuccess)
            return LTE_ERR_CUDA;
        attr_done = true;
    }
    dim3 grid((p.T + TJ - 1) / TJ, p.B * p.H);
    scores_tma_kernel<D, K><<<grid, NT, SMEM, st>>>(tk, tv, p.w, p.bias, z, r, p.H, p.T, status_ptr);
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

int scores_status_fetch_and_clear()
{
    int h = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&h, g_scores_status, sizeof(int)) != cudaSuccess) return -1;
    if (h != 0) cudaMemcpyToSymbol(g_scores_status, &zero, sizeof(int));
    return h;
}

int launch_scores(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    return p.dtype == LTE_BF16 ? by_d<__nv_bfloat16>(p, k, v, z, r, st) : by_d<float>(p, k, v, z, r, st);
}

}  // namespace lte
