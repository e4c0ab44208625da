// Capped retention list (Eq. 5 + "Capped capacity", Section 3.1.3): threshold, then top-R, emitted
// in ascending position order.  One block per (b,h).
//
// Every eligible position j <= T-1-W gets a 32-bit key: 0xFFFFFFFF for sink positions, the monotone
// image of z_j for candidates (z_j > zthr), 0 otherwise.  If more than R keys are non-zero, an exact
// radix select (4 passes of 8 bits, shared-memory histograms) finds the key theta of the R-th largest;
// kept = keys above theta plus the oldest (R - #above) positions whose key equals theta, which is the
// order "z descending, ties to the older token".  A final ordered compaction (ballot prefix sums,
// positions visited in ascending order) writes idx.  Nothing here rounds: the result is exact on z.
#include <cooperative_groups.h>
#include <type_traits>

#include "common.cuh"
#include "select_body.cuh"

namespace lte {
namespace cg = cooperative_groups;
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


// ---- a thread-block cluster per (b,h): long sequences with few heads ---------------------------------------------
// With one block per head a sequence of 32K positions and 16 heads keeps 16 SMs busy for 35 us.  Here CS blocks (a
// cluster) share a head: block `rank` owns the positions [rank, rank + 1) * 512 * KPT, a thread KPT consecutive
// ones in registers.  Block-wide counts become cluster-wide counts by every block writing its total into a slot of
// every block's shared memory (distributed shared memory) followed by one cluster barrier; with only a few keys per
// thread a step settles four bits (fifteen candidate values, fifteen counts), so the upper half of the R-th largest
// key takes 4 exchanges.  The keys that share that upper half go to a short list in the first block's shared
// memory (remote atomics), one warp there settles the lower half, and the result is written back to every block.
// The ordered compaction needs the blocks' (above, equal) totals once more; each block then writes its own segment.
constexpr int kClusterMax = 8;
constexpr int kClusterThreads = 512;                       // two blocks fit an SM, so every cluster of a launch finds room at once
template <int KPT>
__global__ void __launch_bounds__(kClusterThreads, 2) select_cluster_kernel(const float* __restrict__ z, int32_t* __restrict__ idx,
                                                                            int32_t* __restrict__ cnt, int32_t* __restrict__ ncand,
                                                                            int T, int W, int R, int sink, float zthr)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int cs = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    constexpr int NT = kClusterThreads, nwarp = NT / 32, NCNT = 15;
    __shared__ uint32_t s_part[2][NCNT][nwarp];            // warp partials of up to 15 counts (two alternating rows)
    __shared__ uint32_t s_x[2][kClusterMax][16];           // every block's totals, written by the blocks themselves
    __shared__ uint32_t s_wa[32], s_we[32];
    __shared__ uint32_t s_list[kSelList + 3];              // first block: the short list, its length; every block: threshold, need_eq
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int bh = blockIdx.x / cs;
    const float* zz = z + (size_t)bh * T;
    int32_t* out = idx + (size_t)bh * R;
    const int N = T - W > 0 ? T - W : 0;
    const int p0 = (rank * NT + tid) * KPT;
    if (tid == 0) s_list[kSelList] = 0u;
    SELP(0);
    pdl_launch_dependents();
    pdl_wait();                                            // z comes from the previous kernel
    SELP(1);

    uint32_t key[KPT];
    if (KPT % 4 == 0 && (reinterpret_cast<uintptr_t>(zz + p0) & 15u) == 0 && p0 + KPT <= T) {
#pragma unroll
        for (int i = 0; i < KPT; i += 4) {
            const float4 z4 = __ldg(reinterpret_cast<const float4*>(zz + p0 + i));
            key[i] = p0 + i < N ? select_key_from(z4.x, p0 + i, sink, zthr) : 0u;
            key[i + 1] = p0 + i + 1 < N ? select_key_from(z4.y, p0 + i + 1, sink, zthr) : 0u;
            key[i + 2] = p0 + i + 2 < N ? select_key_from(z4.z, p0 + i + 2, sink, zthr) : 0u;
            key[i + 3] = p0 + i + 3 < N ? select_key_from(z4.w, p0 + i + 3, sink, zthr) : 0u;
        }
    } else {
#pragma unroll
        for (int i = 0; i < KPT; ++i) key[i] = p0 + i < N ? select_key_from(__ldg(zz + p0 + i), p0 + i, sink, zthr) : 0u;
    }
    SELP(2);

    // Cluster-wide sums of NC per-thread counts; lane k < NC of every warp returns the k-th total.  A row of s_part and a
    // row of s_x are rewritten two calls later, when every warp (every block) has passed the barrier of the call in
    // between and so has finished reading them.
    int slot = 0;
    auto cluster_sum = [&](auto nc_tag, const uint32_t* c) -> uint32_t {
        constexpr int NC = decltype(nc_tag)::value;
#pragma unroll
        for (int k2 = 0; k2 < NC; ++k2) {
            const uint32_t t = __reduce_add_sync(0xffffffffu, c[k2]);
            if (lane == 0) s_part[slot][k2][wid] = t;
        }
        __syncthreads();
        if (wid == 0) {
            // lane = l: partial sums of count (l % 16) over half of the warps, then the two halves meet
            const int k2 = lane & 15, w0 = (lane >> 4) * (nwarp / 2);
            uint32_t t = 0;
            if (k2 < NC)
                for (int w2 = 0; w2 < nwarp / 2; ++w2) t += s_part[slot][k2][w0 + w2];
            t += __shfl_xor_sync(0xffffffffu, t, 16);
            // the block's NC totals go into this block's row of every block's table: lane l writes count l % 16 to block l / 16 (+ 2, 4, 6)
            for (int r2 = lane >> 4; r2 < cs; r2 += 2)
                if (k2 < NC) *cluster.map_shared_rank(&s_x[slot][rank][k2], r2) = t;
        }
        cluster.sync();
        uint32_t tot = 0;
        if (lane < NC)
            for (int r2 = 0; r2 < cs; ++r2) tot += s_x[slot][r2][lane];
        slot ^= 1;
        return tot;
    };
    using One = std::integral_constant<int, 1>;
    using Two = std::integral_constant<int, 2>;
    using Fifteen = std::integral_constant<int, 15>;

    uint32_t c1[1] = {0};
#pragma unroll
    for (int i = 0; i < KPT; ++i) c1[0] += key[i] != 0u;
    const uint32_t nc = __shfl_sync(0xffffffffu, cluster_sum(One{}, c1), 0);
    SELP(3);
    if (rank == 0 && tid == 0 && ncand) ncand[bh] = (int32_t)nc;

    uint32_t theta = 0, need_eq = 0;
    if (R > 0 && nc > (uint32_t)R) {
        uint32_t prefix = 0;
        // four bits per exchange: the largest d in 1..15 such that at least R keys reach prefix | d << b (0: none does).
        // The counts fall with d, so d is the number of counts that reach R.
        auto four_bits = [&](int b) {
            uint32_t n[15];
#pragma unroll
            for (int d = 0; d < 15; ++d) n[d] = 0;
#pragma unroll
            for (int i = 0; i < KPT; ++i)
#pragma unroll
                for (int d = 0; d < 15; ++d) n[d] += key[i] >= (prefix | ((uint32_t)(d + 1) << b));
            const uint32_t tot = cluster_sum(Fifteen{}, n);
            const uint32_t d = (uint32_t)__popc(__ballot_sync(0xffffffffu, lane < 15 && tot >= (uint32_t)R));
            prefix |= d << b;
        };
        for (int b = 28; b >= 16; b -= 4) four_bits(b);
        SELP(4);
        // keys above the upper half, keys sharing it
        const uint32_t hi = prefix >> 16;
        uint32_t c2[2] = {0, 0};
#pragma unroll
        for (int i = 0; i < KPT; ++i) { c2[0] += (key[i] >> 16) > hi; c2[1] += (key[i] >> 16) == hi; }
        const uint32_t am = cluster_sum(Two{}, c2);
        const uint32_t above = __shfl_sync(0xffffffffu, am, 0), match = __shfl_sync(0xffffffffu, am, 1);
        SELP(7);
        if (match <= (uint32_t)kSelList) {
            uint32_t* list0 = cluster.map_shared_rank(&s_list[0], 0);
#pragma unroll
            for (int i = 0; i < KPT; ++i)
                if ((key[i] >> 16) == hi) list0[atomicAdd(&list0[kSelList], 1u)] = key[i];
            cluster.sync();
            SELP(8);
            if (rank == 0 && wid == 0) {
                uint32_t pf = prefix, g;
                if (match <= 32u) {
                    // the usual case: one key per lane, a vote per bit
                    const uint32_t mine = (uint32_t)lane < match ? s_list[lane] : 0u;   // 0 never counts: candidates are > 0
                    for (int b2 = 15; b2 >= 0; --b2) {
                        const uint32_t cand = pf | (1u << b2);
                        if (above + (uint32_t)__popc(__ballot_sync(0xffffffffu, mine >= cand)) >= (uint32_t)R) pf = cand;
                    }
                    g = above + (uint32_t)__popc(__ballot_sync(0xffffffffu, mine > pf));
                } else {
                    for (int b2 = 15; b2 >= 0; --b2) {
                        const uint32_t cand = pf | (1u << b2);
                        uint32_t c = 0;
                        for (uint32_t l = lane; l < match; l += 32) c += s_list[l] >= cand;
                        if (above + __reduce_add_sync(0xffffffffu, c) >= (uint32_t)R) pf = cand;
                    }
                    uint32_t c = 0;                        // keys strictly above the threshold: all of them are in `above` or the list
                    for (uint32_t l = lane; l < match; l += 32) c += s_list[l] > pf;
                    g = above + __reduce_add_sync(0xffffffffu, c);
                }
                if (lane < cs) {
                    uint32_t* dst = cluster.map_shared_rank(&s_list[kSelList + 1], lane);
                    dst[0] = pf; dst[1] = (uint32_t)R - g;
                }
            }
            cluster.sync();
            SELP(9);
            theta = s_list[kSelList + 1];
            need_eq = s_list[kSelList + 2];
        } else {
            for (int b = 12; b >= 0; b -= 4) four_bits(b);
            theta = prefix;
            uint32_t g1[1] = {0};
#pragma unroll
            for (int i = 0; i < KPT; ++i) g1[0] += key[i] > theta;
            need_eq = (uint32_t)R - __shfl_sync(0xffffffffu, cluster_sum(One{}, g1), 0);
        }
    }
    SELP(5);
    // ---- ordered compaction: exclusive scan of (above, equal) counts over the threads' segments, blocks in rank order
    uint32_t a = 0, e = 0;
    if (R > 0) {
#pragma unroll
        for (int i = 0; i < KPT; ++i) { a += key[i] > theta; e += (need_eq > 0 && key[i] == theta && p0 + i < N); }
    }
    uint32_t ia = a, ie = e;                               // inclusive warp scans
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t ta = __shfl_up_sync(0xffffffffu, ia, o), te = __shfl_up_sync(0xffffffffu, ie, o);
        if (lane >= o) { ia += ta; ie += te; }
    }
    if (lane == 31) { s_wa[wid] = ia; s_we[wid] = ie; }
    __syncthreads();
    if (wid == 0) {
        const uint32_t wa = lane < nwarp ? s_wa[lane] : 0u, we = lane < nwarp ? s_we[lane] : 0u;
        uint32_t xa = wa, xe = we;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t ta = __shfl_up_sync(0xffffffffu, xa, o), te = __shfl_up_sync(0xffffffffu, xe, o);
            if (lane >= o) { xa += ta; xe += te; }
        }
        s_wa[lane] = xa - wa; s_we[lane] = xe - we;        // exclusive warp offsets
        const uint32_t ta = __shfl_sync(0xffffffffu, xa, 31), te = __shfl_sync(0xffffffffu, xe, 31);   // this block's totals
        if (lane < cs) {
            uint32_t* dst = cluster.map_shared_rank(&s_x[slot][rank][0], lane);
            dst[0] = ta; dst[1] = te;
        }
    }
    cluster.sync();
    uint32_t a_before = s_wa[wid] + ia - a, e_before = s_we[wid] + ie - e;
    for (int r2 = 0; r2 < rank; ++r2) { a_before += s_x[slot][r2][0]; e_before += s_x[slot][r2][1]; }
    if (R > 0) {
#pragma unroll
        for (int i = 0; i < KPT; ++i) {
            const bool above = key[i] > theta;
            const bool equal = need_eq > 0 && key[i] == theta && p0 + i < N;
            if (above || (equal && e_before < need_eq)) {
                const uint32_t sl = a_before + (e_before < need_eq ? e_before : need_eq);
                if (sl < (uint32_t)R) out[sl] = p0 + i;
            }
            a_before += above; e_before += equal;
        }
    }
    const uint32_t kept = R > 0 ? (nc < (uint32_t)R ? nc : (uint32_t)R) : 0u;
    for (int i = (int)kept + rank * NT + tid; i < R; i += cs * NT) out[i] = -1;
    if (rank == 0 && tid == 0) cnt[bh] = (int32_t)kept;
    cluster.sync();                                        // no block leaves while another may still read its shared memory
    SELP(6);
}

template <int KPT>
cudaError_t launch_select_cluster(int BH, int cs, cudaStream_t st, const float* z, int32_t* idx, int32_t* cnt, int32_t* ncand,
                                  int T, int W, int R, int sink, float zthr)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(BH * cs);
    cfg.blockDim = dim3(kClusterThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, select_cluster_kernel<KPT>, z, idx, cnt, ncand, T, W, R, sink, zthr);
}

}  // namespace

int launch_select(const Params& p, const float* z, int32_t* idx, int32_t* cnt, int32_t* ncand, cudaStream_t st)
{
    const int N = p.T - p.W > 0 ? p.T - p.W : 0;
    {
        // long sequences, few heads: a cluster of blocks per head (every cluster resident at once)
        int sms = 0;
        if (int e = device_sm_count(&sms)) return e;
        const int BH = p.B * p.H;
        if (N >= 16384 && N <= kClusterMax * kClusterThreads * 16 && BH * kClusterMax <= sms) {
            const int kpt = (N + kClusterMax * kClusterThreads - 1) / (kClusterMax * kClusterThreads);
            cudaError_t e;
            if (kpt <= 8) e = launch_select_cluster<8>(BH, kClusterMax, st, z, idx, cnt, ncand, p.T, p.W, p.R, p.sink, p.zthr);
            else e = launch_select_cluster<16>(BH, kClusterMax, st, z, idx, cnt, ncand, p.T, p.W, p.R, p.sink, p.zthr);
            return cuda_status(e);
        }
    }
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
