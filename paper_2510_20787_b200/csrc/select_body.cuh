// Capped selection of one (b,h) by a group of threads that keep their keys in registers (Section 3.1.3, "Capped
// capacity"): the body of the select kernel, written for any group of whole warps with a barrier of its own.
//
// Thread `tid` of `nthr` owns KPT consecutive positions.  The R-th largest key is found by bisection on its 32 bits:
// each step counts the keys >= a candidate value (compares in registers, a warp reduction, one group barrier), so
// there is no histogram and no contention however concentrated the logits are.  The ordered compaction is one
// group-wide exclusive scan of the per-thread (above, equal) counts, after which each thread writes the kept
// positions of its own segment.  `sync` is the group's barrier; s_part [2][32], s_wa [32], s_we [32] are its scratch.
#pragma once
#include "common.cuh"

namespace lte {

#ifdef LTE_PROFILE
__device__ long long g_selprof[16];
#define SELP(i) do { if (blockIdx.x == 0 && tid == 0) { g_selprof[i] = clock64(); if ((i) == 0 || (i) == 6) { unsigned long long gt; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt)); g_selprof[(i) == 0 ? 10 : 11] = (long long)gt; } } } while (0)
#else
#define SELP(i) do {} while (0)
#endif

// key of position j: 0xFFFFFFFF for sink positions, the monotone image of z_j for candidates (z_j > zthr), 0 otherwise.
__device__ __forceinline__ uint32_t select_key_from(float z, int j, int sink, float zthr) {
    if (j < sink) return 0xFFFFFFFFu;
    return z > zthr ? order_key(z) : 0u;
}

constexpr int kSelList = 1024;      // keys that share the upper half of the threshold: up to this many are settled by one warp

template <int KPT, typename Sync>
__device__ __forceinline__ void select_group(const float* __restrict__ zz, int32_t* __restrict__ out, int32_t* cnt_out,
                                             int32_t* ncand_out, int T, int W, int R, int sink, float zthr, int tid,
                                             int nthr, uint32_t (*s_part)[32], uint32_t* s_wa, uint32_t* s_we, Sync sync,
                                             uint32_t* s_list = nullptr)
{
    const int lane = tid & 31, wid = tid >> 5, nwarp = nthr >> 5;
    const int N = T - W > 0 ? T - W : 0;
    const int p0 = tid * KPT;

    // A thread's KPT consecutive logits are one run of memory: 16-byte loads through L1 where the run is aligned (a thread's
    // loads then touch each 32-byte sector once: scalar loads past L1 made this phase 17 us of 36 at 32K positions per head)
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
    // block-wide sum of a per-thread count, one barrier per call and no atomics: every warp leaves its sum in one of two
    // alternating rows of partials, and after the barrier every warp adds the row up itself.  A row is rewritten two calls
    // later, when every warp has passed the barrier of the call in between and so has finished reading it.
    int slot = 0;
    auto block_sum = [&](uint32_t c) -> uint32_t {
        c = __reduce_add_sync(0xffffffffu, c);
        if (lane == 0) s_part[slot][wid] = c;
        sync();
        const uint32_t total = __reduce_add_sync(0xffffffffu, lane < nwarp ? s_part[slot][lane] : 0u);
        slot ^= 1;
        return total;
    };
    SELP(2);
    if (tid == 0 && s_list != nullptr) s_list[kSelList] = 0u;   // the first group barrier below publishes it
    uint32_t c0 = 0;
#pragma unroll
    for (int i = 0; i < KPT; ++i) c0 += key[i] != 0u;
    const uint32_t nc = block_sum(c0);
    if (tid == 0 && ncand_out) *ncand_out = (int32_t)nc;

    SELP(3);
    uint32_t theta = 0, need_eq = 0;
    if (R > 0 && nc > (uint32_t)R) {
        uint32_t prefix = 0;
        int bit = 31;
        for (; bit >= 16; --bit) {
            const uint32_t cand = prefix | (1u << bit);
            uint32_t c = 0;
#pragma unroll
            for (int i = 0; i < KPT; ++i) c += key[i] >= cand;
            if (block_sum(c) >= (uint32_t)R) prefix = cand;  // at least R keys are >= cand: the R-th largest is too
        }
        // The upper half of the R-th largest key is known.  Only the keys that share it can still move a count, and with
        // spread-out logits they are few: they go into a short list, and one warp settles the lower 16 bits on it without
        // any group barrier.  (s_list: kSelList entries, then the list length, the threshold and the number of keys equal to it to keep.)
        SELP(4);
        bool done = false;
        bool have_need = false;
        if (s_list != nullptr && N < 65536) {
            const uint32_t hi = prefix >> 16;
            uint32_t cam = 0;                                  // keys above the upper half (low 16 bits of the sum), keys sharing it (high)
#pragma unroll
            for (int i = 0; i < KPT; ++i) cam += ((key[i] >> 16) > hi ? 1u : 0u) + ((key[i] >> 16) == hi ? 65536u : 0u);
            const uint32_t both = block_sum(cam);
            const uint32_t above = both & 0xffffu, match = both >> 16;
            SELP(7);
            if (match <= (uint32_t)kSelList) {
                // (the list length was zeroed before the first group barrier of this function)
#pragma unroll
                for (int i = 0; i < KPT; ++i)
                    if ((key[i] >> 16) == hi) s_list[atomicAdd(&s_list[kSelList], 1u)] = key[i];
                sync();
                SELP(8);
                if (wid == 0) {
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
                    if (lane == 0) { s_list[kSelList + 1] = pf; s_list[kSelList + 2] = (uint32_t)R - g; }
                }
                sync();
                SELP(9);
                prefix = s_list[kSelList + 1];
                need_eq = s_list[kSelList + 2];
                done = true; have_need = true;
            }
        }
        if (!done) {
            for (; bit >= 0; --bit) {
                const uint32_t cand = prefix | (1u << bit);
                uint32_t c = 0;
#pragma unroll
                for (int i = 0; i < KPT; ++i) c += key[i] >= cand;
                if (block_sum(c) >= (uint32_t)R) prefix = cand;
            }
        }
        theta = prefix;
        if (!have_need) {
            uint32_t g = 0;
#pragma unroll
            for (int i = 0; i < KPT; ++i) g += key[i] > theta;
            need_eq = (uint32_t)R - block_sum(g);
        }
    }
    SELP(5);
    // ---- ordered compaction: exclusive scan of (above, equal) counts over the threads' segments
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
    sync();
    if (wid == 0) {
        uint32_t wa = lane < nwarp ? s_wa[lane] : 0u, we = lane < nwarp ? s_we[lane] : 0u;
        uint32_t xa = wa, xe = we;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t ta = __shfl_up_sync(0xffffffffu, xa, o), te = __shfl_up_sync(0xffffffffu, xe, o);
            if (lane >= o) { xa += ta; xe += te; }
        }
        s_wa[lane] = xa - wa; s_we[lane] = xe - we;        // exclusive warp offsets
    }
    sync();
    uint32_t a_before = s_wa[wid] + ia - a, e_before = s_we[wid] + ie - e;
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
    for (int i = (int)kept + tid; i < R; i += nthr) out[i] = -1;
    if (tid == 0) *cnt_out = (int32_t)kept;
    SELP(6);
}

}  // namespace lte
