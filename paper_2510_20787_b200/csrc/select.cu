// Capped retention list (Eq. 5 + "Capped capacity", Section 3.1.3): threshold, then top-R, emitted
// in ascending position order.  One block per (b,h).
//
// Every eligible position j <= T-1-W gets a 32-bit key: 0xFFFFFFFF for sink positions, the monotone
// image of z_j for candidates (z_j > zthr), 0 otherwise.  If more than R keys are non-zero, an exact
// radix select (4 passes of 8 bits, shared-memory histograms) finds the key theta of the R-th largest;
// kept = keys above theta plus the oldest (R - #above) positions whose key equals theta, which is the
// order "z descending, ties to the older token".  A final ordered compaction (ballot prefix sums,
// positions visited in ascending order) writes idx.  Nothing here rounds: the result is exact on z.
#include "common.cuh"
#include "select_body.cuh"

namespace lte {
namespace {

__device__ __forceinline__ uint32_t key_of(const float* zz, int j, int sink, float zthr) {
    if (j < sink) return 0xFFFFFFFFu;
    float z = zz[j];
    return z > zthr ? order_key(z) : 0u;
}

// CACHED: the keys of all eligible positions are computed once and kept in dynamic shared memory, so the radix passes
// and the compaction never go back to L2; otherwise every pass recomputes them from z.
template <bool CACHED>
__global__ void select_kernel(const float* __restrict__ z, int32_t* __restrict__ idx, int32_t* __restrict__ cnt,
                              int32_t* __restrict__ ncand, int T, int W, int R, int sink, float zthr)
{
    extern __shared__ uint32_t s_keys[];
    __shared__ uint32_t hist[256];
    __shared__ uint32_t warp_tot[2][32];
    __shared__ uint32_t sh_prefix, sh_remaining, sh_ncand;

    const int bh = blockIdx.x;
    const float* zz = z + (size_t)bh * T;
    int32_t* out = idx + (size_t)bh * R;
    const int N = T - W > 0 ? T - W : 0;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int lane = tid & 31, wid = tid >> 5, nwarp = nthr >> 5;

    auto key_at = [&](int j) -> uint32_t { return CACHED ? s_keys[j] : key_of(zz, j, sink, zthr); };
    // ---- pass 0: number of candidates (and the key cache)
    if (tid == 0) sh_ncand = 0;
    __syncthreads();
    {
        uint32_t c = 0;
        for (int j = tid; j < N; j += nthr) {
            const uint32_t key = key_of(zz, j, sink, zthr);
            if (CACHED) s_keys[j] = key;
            c += key != 0u;
        }
        c = __reduce_add_sync(0xffffffffu, c);
        if (lane == 0 && c) atomicAdd(&sh_ncand, c);
    }
    __syncthreads();
    const uint32_t nc = sh_ncand;
    if (tid == 0 && ncand) ncand[bh] = (int32_t)nc;

    uint32_t theta = 0, need_eq = 0;
    if (R > 0 && nc > (uint32_t)R) {
        if (tid == 0) { sh_prefix = 0; sh_remaining = (uint32_t)R; }
        uint32_t mask = 0;
        for (int shift = 24; shift >= 0; shift -= 8) {
            for (int i = tid; i < 256; i += nthr) hist[i] = 0;
            __syncthreads();
            const uint32_t prefix = sh_prefix;
            for (int j0 = 0; j0 < N; j0 += nthr) {
                const int j = j0 + tid;
                uint32_t key = j < N ? key_at(j) : 0u;
                const bool in = j < N && (key & mask) == prefix;
                const uint32_t dig = in ? (key >> shift) & 255u : 0xFFFFFFFFu;
                const uint32_t peers = __match_any_sync(0xffffffffu, dig);
                if (in && lane == __ffs(peers) - 1) atomicAdd(&hist[dig], (uint32_t)__popc(peers));
            }
            __syncthreads();
            if (wid == 0) {
                // lane l owns digits 255-8l .. 248-8l (descending); find the digit holding rank `remaining`
                uint32_t loc[8], s = 0;
#pragma unroll
                for (int u = 0; u < 8; ++u) { loc[u] = hist[255 - 8 * lane - u]; s += loc[u]; }
                uint32_t incl = s;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += t;
                }
                const uint32_t rem = sh_remaining;
                __syncwarp();
                const uint32_t before = incl - s;
                if (before < rem && rem <= incl) {          // exactly one lane owns the rank
                    uint32_t b = before;
                    bool done = false;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (!done && rem <= b + loc[u]) {
                            sh_prefix = prefix | ((uint32_t)(255 - 8 * lane - u) << shift);
                            sh_remaining = rem - b;
                            done = true;
                        }
                        b += loc[u];
                    }
                }
            }
            mask |= 255u << shift;
            __syncthreads();
        }
        theta = sh_prefix;
        need_eq = sh_remaining;
    }
    // nc <= R (or R == 0): theta = 0, need_eq = 0 keeps exactly the non-zero keys (none if R == 0)

    // ---- ordered compaction
    uint32_t runA = 0, runE = 0;     // kept-above and equal-to-theta counts before this chunk
    int buf = 0;
    for (int j0 = 0; j0 < N && R > 0; j0 += nthr, buf ^= 1) {
        const int j = j0 + tid;
        const uint32_t key = j < N ? key_at(j) : 0u;
        const bool above = key > theta;
        const bool equal = need_eq > 0 && key == theta && j < N;
        const uint32_t bA = __ballot_sync(0xffffffffu, above), bE = __ballot_sync(0xffffffffu, equal);
        if (lane == 0) warp_tot[buf][wid] = (uint32_t)__popc(bA) | ((uint32_t)__popc(bE) << 16);
        __syncthreads();
        uint32_t preA = 0, preE = 0, totA = 0, totE = 0;
        for (int w2 = 0; w2 < nwarp; ++w2) {
            const uint32_t t = warp_tot[buf][w2];
            if (w2 < wid) { preA += t & 0xffffu; preE += t >> 16; }
            totA += t & 0xffffu; totE += t >> 16;
        }
        const uint32_t lt = (1u << lane) - 1u;
        const uint32_t a_before = runA + preA + (uint32_t)__popc(bA & lt);
        const uint32_t e_before = runE + preE + (uint32_t)__popc(bE & lt);
        if (above || (equal && e_before < need_eq)) {
            const uint32_t slot = a_before + (e_before < need_eq ? e_before : need_eq);
            if (slot < (uint32_t)R) out[slot] = j;
        }
        runA += totA; runE += totE;
    }
    const uint32_t kept = R > 0 ? (nc < (uint32_t)R ? nc : (uint32_t)R) : 0u;
    for (int i = (int)kept + tid; i < R; i += nthr) out[i] = -1;
    if (tid == 0) cnt[bh] = (int32_t)kept;
}


// ---- register-resident variant: every thread keeps KPT consecutive keys in registers ---------------------------------
// The R-th largest key is found by bisection on its 32 bits: each step counts the keys >= a candidate value (compares
// in registers, one shared-memory atomic per warp, one block barrier), so there is no histogram and no contention
// however concentrated the logits are.  The ordered compaction is one block-wide exclusive scan of the per-thread
// (above, equal) counts, after which each thread writes the kept positions of its own segment.
template <int KPT>
__global__ void __launch_bounds__(1024) select_reg_kernel(const float* __restrict__ z, int32_t* __restrict__ idx,
                                                          int32_t* __restrict__ cnt, int32_t* __restrict__ ncand, int T,
                                                          int W, int R, int sink, float zthr)
{
    __shared__ uint32_t s_part[2][32];
    __shared__ uint32_t s_wa[32], s_we[32];
    __shared__ uint32_t s_list[kSelList + 3];
    const int tid = threadIdx.x;
    SELP(0);
    pdl_launch_dependents();
    pdl_wait();                                            // z comes from the previous kernel
    SELP(1);
    const int bh = blockIdx.x;
    select_group<KPT>(z + (size_t)bh * T, idx + (size_t)bh * R, cnt + bh, ncand ? ncand + bh : nullptr, T, W, R, sink, zthr,
                      (int)threadIdx.x, (int)blockDim.x, s_part, s_wa, s_we, [] { __syncthreads(); }, s_list);
}

}  // namespace

int launch_select(const Params& p, const float* z, int32_t* idx, int32_t* cnt, int32_t* ncand, cudaStream_t st)
{
    const int N = p.T - p.W > 0 ? p.T - p.W : 0;
    {
        // register-resident kernel: up to 64 keys per thread
        const int nt = N <= 2048 ? 256 : 1024;
        const int kpt = (N + nt - 1) / nt;
        const int BH = p.B * p.H;
#define LTE_SEL(KPT) launch_pdl(select_reg_kernel<KPT>, dim3(BH), dim3(nt), 0, st, z, idx, cnt, ncand, p.T, p.W, p.R, p.sink, p.zthr)
        if (kpt <= 64) {
            if (kpt <= 1) LTE_SEL(1); else if (kpt <= 2) LTE_SEL(2); else if (kpt <= 4) LTE_SEL(4);
            else if (kpt <= 8) LTE_SEL(8); else if (kpt <= 16) LTE_SEL(16); else if (kpt <= 32) LTE_SEL(32);
            else LTE_SEL(64);
            return cuda_status(cudaGetLastError());
        }
#undef LTE_SEL
    }
    const int threads = N <= 1024 ? 256 : (N <= 4096 ? 512 : 1024);
    const size_t key_bytes = (size_t)N * 4;
    constexpr size_t kCacheMax = 200 * 1024;              // keys of up to 51200 positions stay on chip
    if (key_bytes <= kCacheMax) {
        static PerDeviceOnce attr;
        if (int e = attr.run([] { return cudaFuncSetAttribute(select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCacheMax); }))
            return e;
        select_kernel<true><<<p.B * p.H, threads, key_bytes, st>>>(z, idx, cnt, ncand, p.T, p.W, p.R, p.sink, p.zthr);
    } else {
        select_kernel<false><<<p.B * p.H, threads, 0, st>>>(z, idx, cnt, ncand, p.T, p.W, p.R, p.sink, p.zthr);
    }
    return cuda_status(cudaGetLastError());
}

}  // namespace lte

#ifdef LTE_PROFILE
extern "C" int lte_selprof_read(long long* out)
{
    return cudaMemcpyFromSymbol(out, lte::g_selprof, sizeof(long long) * 16) == cudaSuccess ? 0 : -1;
}
#endif
