// Training-side statistics of the scorer (Section 3.1.2, Eq. 7; Algorithm 1): per head the number of tokens whose
// retention score passes the threshold, averaged over the batch, and the value of the sparsity penalty
// sum_h lambda_h sum_{b,i} ReLU(r - tau).  Two kernels, both with a fixed summation order (no floating-point atomics).
#include "common.cuh"

namespace lte {
namespace {

constexpr int ST = 256;

// block per (b,h): count and penalty sum of one sequence
__global__ void __launch_bounds__(ST) stats_partial_kernel(const float* __restrict__ z, float* __restrict__ part, int Tlen, float zthr,
                                                           float tau)
{
    __shared__ float s_c[ST / 32], s_p[ST / 32];
    const int bh = blockIdx.x, tid = threadIdx.x;
    const float* zr = z + (size_t)bh * Tlen;
    float c = 0.f, p = 0.f;
    for (int i = tid; i < Tlen; i += ST) {
        const float zi = zr[i];
        if (zi > zthr) {                                       // r > tau  <=>  z > logit(tau), the test the selection uses
            c += 1.f;
            p += fmaxf(1.f / (1.f + __expf(-zi)) - tau, 0.f);
        }
    }
    c = warp_sum(c); p = warp_sum(p);
    if ((tid & 31) == 0) { s_c[tid >> 5] = c; s_p[tid >> 5] = p; }
    __syncthreads();
    if (tid == 0) {
        float cc = 0.f, pp = 0.f;
        for (int w = 0; w < ST / 32; ++w) { cc += s_c[w]; pp += s_p[w]; }
        part[2 * (size_t)bh] = cc;
        part[2 * (size_t)bh + 1] = pp;
    }
}

// one block: count[h] = mean over b; penalty = sum_h lambda_h sum_b (in index order)
__global__ void stats_final_kernel(const float* __restrict__ part, const float* __restrict__ lambda, float* __restrict__ count,
                                   float* __restrict__ penalty, int B, int H)
{
    extern __shared__ float s_pen[];                           // [H]
    for (int h = threadIdx.x; h < H; h += blockDim.x) {
        float cc = 0.f, pp = 0.f;
        for (int b = 0; b < B; ++b) { cc += part[2 * ((size_t)b * H + h)]; pp += part[2 * ((size_t)b * H + h) + 1]; }
        count[h] = cc / (float)B;
        s_pen[h] = (lambda ? lambda[h] : 1.f) * pp;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int h = 0; h < H; ++h) t += s_pen[h];
        *penalty = t;
    }
}

}  // namespace

int launch_sparsity_stats(const Params& p, const float* z, const float* lambda, float* count, float* penalty, float* part, float tau,
                          cudaStream_t st)
{
    stats_partial_kernel<<<p.B * p.H, ST, 0, st>>>(z, part, p.T, p.zthr, tau);
    if (cudaGetLastError() != cudaSuccess) return LTE_ERR_CUDA;
    stats_final_kernel<<<1, 256, (size_t)p.H * sizeof(float), st>>>(part, lambda, count, penalty, p.B, p.H);
    return cuda_status(cudaGetLastError());
}

}  // namespace lte
