// Chunked (continued) prefill on top of a decode cache (Section 3.1.3, "Cached prefilling and decoding"): glue kernels.
//
// The cache holds n0 tokens: a ring with the last min(n0, W) of them and a pool of retained ones.  A chunk of Tc tokens
// arrives.  The chunk-end reading: the pool entries compete with the tokens that leave the window while the chunk
// arrives, the best R form the new list, and query i of the chunk sees its window plus the list entries older than its
// window.  This is what the one-shot prefill computes over the "local sequence"
//     rows [0, R0)            the pool rows, slot order      (R0 = R once anything has left the window, else 0)
//     rows [R0, R0 + Wn)      the ring in time order         (Wn = min(n0, W))
//     rows [R0 + Wn, T_loc)   the chunk
// because every pool row is older than every chunk query's window and the window of a chunk query never reaches below
// row R0.  So the path is: gather the local sequence (here), score it (the scorer kernels), merge the logits the cache
// already holds (here), select, attend (the prefill kernels, told that their queries start at row R0 + Wn), and write the
// new cache (here).  Local row r stands for position pos(r) = old pool position (r < R0) or n0 - Wn + (r - R0).
#include "common.cuh"

namespace lte {

__device__ StatusWord g_chunk_status = LTE_STATUS_INIT;   // report only; 31: the cache does not hold n_past tokens

namespace {

// one 16-byte piece of a cache row -> the same piece of a plain row (the swizzled layout permutes the pieces of a row)
__device__ __forceinline__ int piece_src(const CacheLayout& L, int row, int c) { return L.swz ? (c ^ (row & 7)) : c; }

constexpr int kRowsPerBlock = 128;

// Block (part, (b,h)): rows [part 128, part 128 + 128) of the local sequence: pool rows, ring rows (time order) and the
// chunk's rows of k, v.  Part 0 also copies the logits of the pool and the ring into zsrc [R0 + Wn] and the pool's
// positions into oldpos [R], and writes gate[b,h] = 1 if the head's cache holds n0 tokens as the call said, else 0 (the
// head's cache is then left alone by the commit of this same call; the flag lives in the call's scratch, so it says
// nothing about any other call).
__global__ void chunk_gather_kernel(const unsigned char* __restrict__ cache, CacheLayout L, const unsigned char* __restrict__ kc,
                                    const unsigned char* __restrict__ vc, unsigned char* __restrict__ klin,
                                    unsigned char* __restrict__ vlin, float* __restrict__ zsrc, int32_t* __restrict__ oldpos,
                                    int32_t* __restrict__ gate, int D, int W, int R, int n0, int R0, int Wn, int Tloc)
{
    const int bh = blockIdx.y;
    const unsigned char* blk = cache + L.header + (size_t)bh * L.stride;
    const uint4* Kc = reinterpret_cast<const uint4*>(blk + L.off_k);
    const uint4* Vc = reinterpret_cast<const uint4*>(blk + L.off_v);
    const float* zc = reinterpret_cast<const float*>(blk + L.off_z);
    const int32_t* pidx = reinterpret_cast<const int32_t*>(blk + L.off_pidx);
    const int32_t* meta = reinterpret_cast<const int32_t*>(blk + L.off_meta);
    if (meta[0] != n0) {
        if (threadIdx.x == 0) { atomicExch(&g_chunk_status.code, 31); if (blockIdx.x == 0) gate[bh] = 0; }
        return;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) gate[bh] = 1;
    const int cnt = meta[1];
    const int pieces = D * (int)L.esz / 16;                    // 16-byte pieces per row
    uint4* kd = reinterpret_cast<uint4*>(klin) + (size_t)bh * Tloc * pieces;
    uint4* vd = reinterpret_cast<uint4*>(vlin) + (size_t)bh * Tloc * pieces;
    const int rows = R0 + Wn, Tc = Tloc - rows;
    const uint4* kq = reinterpret_cast<const uint4*>(kc) + (size_t)bh * Tc * pieces;
    const uint4* vq = reinterpret_cast<const uint4*>(vc) + (size_t)bh * Tc * pieces;
    const int r_lo = blockIdx.x * kRowsPerBlock, r_hi = min(r_lo + kRowsPerBlock, Tloc);
    for (int e = r_lo * pieces + threadIdx.x; e < r_hi * pieces; e += blockDim.x) {
        const int r = e / pieces, c = e % pieces;
        uint4 kx = make_uint4(0, 0, 0, 0), vx = kx;
        if (r >= rows) {
            kx = kq[(size_t)(r - rows) * pieces + c];
            vx = vq[(size_t)(r - rows) * pieces + c];
        } else {
            int src = -1;
            if (r < R0) { if (r < cnt) src = W + r; }
            else src = (n0 - Wn + (r - R0)) % W;
            if (src >= 0) {
                const int cs = piece_src(L, src, c);
                kx = Kc[(size_t)src * pieces + cs];
                vx = Vc[(size_t)src * pieces + cs];
            }
        }
        kd[(size_t)r * pieces + c] = kx;
        vd[(size_t)r * pieces + c] = vx;
    }
    if (blockIdx.x != 0) return;
    for (int r = threadIdx.x; r < rows; r += blockDim.x) {
        float zz = -INFINITY;
        if (r < R0) { if (r < cnt) zz = zc[W + r]; }
        else zz = zc[(n0 - Wn + (r - R0)) % W];
        zsrc[(size_t)bh * (R + W) + r] = zz;
    }
    for (int r = threadIdx.x; r < R; r += blockDim.x) oldpos[(size_t)bh * R + r] = r < cnt ? pidx[r] : -1;
}

// Logits of the local sequence.  In: z = the scorer's output over the local sequence (wrong where the receptive field
// reaches below row R0 + half, undefined for the pool rows).  Out: z = the logit of each row's token (the cache's own where
// it holds one), zrank = the same with sink tokens lifted to +inf, which is what the selection ranks by.
__global__ void chunk_merge_z_kernel(float* __restrict__ z, float* __restrict__ zrank, const float* __restrict__ zsrc,
                                     const int32_t* __restrict__ oldpos, int R, int W, int n0, int R0, int Wn, int Tloc,
                                     int half, int sink)
{
    const int bh = blockIdx.y;
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= Tloc) return;
    float zt;
    int pos;
    if (r < R0) {
        pos = oldpos[(size_t)bh * R + r];
        zt = zsrc[(size_t)bh * (R + W) + r];
        if (pos < 0) zt = -INFINITY;
    } else {
        pos = n0 - Wn + (r - R0);
        zt = z[(size_t)bh * Tloc + r];
        if (r < R0 + Wn) {
            const float zc = zsrc[(size_t)bh * (R + W) + r];
            // a ring token keeps the logit the cache holds; one the cache has not scored yet is scored now, unless its
            // left neighbours are no longer there (then it stays unscored, as in the decode step)
            if (zc > -INFINITY) zt = zc;
            else if (R0 > 0 && r < R0 + half) zt = -INFINITY;
        }
    }
    z[(size_t)bh * Tloc + r] = zt;
    zrank[(size_t)bh * Tloc + r] = (pos >= 0 && pos < sink) ? INFINITY : zt;
}

// Block (part, (b,h)): the cache after the chunk, 128 of its key/value rows per part; part 0 also writes the logits, the
// positions and the counters.  Ring <- the last min(n1, W) rows of the local sequence, pool <- the rows the
// selection kept, with their logits and positions.  Reads only the scratch copies, so the old block can be overwritten.
__global__ void chunk_commit_kernel(unsigned char* __restrict__ cache, CacheLayout L, const unsigned char* __restrict__ klin,
                                    const unsigned char* __restrict__ vlin, const float* __restrict__ z,
                                    const int32_t* __restrict__ idx, const int32_t* __restrict__ cntp,
                                    const int32_t* __restrict__ oldpos, const int32_t* __restrict__ gate, int D, int W, int R,
                                    int n0, int n1, int R0, int Wn, int Tloc, int half)
{
    const int bh = blockIdx.y;
    if (gate[bh] == 0) return;                                 // this call's gather found another state: leave the cache alone
    unsigned char* blk = cache + L.header + (size_t)bh * L.stride;
    uint4* Kc = reinterpret_cast<uint4*>(blk + L.off_k);
    uint4* Vc = reinterpret_cast<uint4*>(blk + L.off_v);
    float* zc = reinterpret_cast<float*>(blk + L.off_z);
    int32_t* pidx = reinterpret_cast<int32_t*>(blk + L.off_pidx);
    int32_t* meta = reinterpret_cast<int32_t*>(blk + L.off_meta);
    const int pieces = D * (int)L.esz / 16;
    const uint4* ks = reinterpret_cast<const uint4*>(klin) + (size_t)bh * Tloc * pieces;
    const uint4* vs = reinterpret_cast<const uint4*>(vlin) + (size_t)bh * Tloc * pieces;
    const float* zl = z + (size_t)bh * Tloc;
    const int Wnew = n1 < W ? n1 : W;
    const int cnt = R > 0 ? cntp[bh] : 0;
    const int a_lo = blockIdx.x * kRowsPerBlock, a_hi = min(a_lo + kRowsPerBlock, Wnew + cnt);
    for (int e = a_lo * pieces + threadIdx.x; e < a_hi * pieces; e += blockDim.x) {
        const int a = e / pieces, c = e % pieces;
        int r, row;
        if (a < Wnew) { r = Tloc - Wnew + a; row = (n1 - Wnew + a) % W; }
        else { r = idx[(size_t)bh * R + (a - Wnew)]; row = W + (a - Wnew); }
        const int cd = piece_src(L, row, c);
        Kc[(size_t)row * pieces + cd] = ks[(size_t)r * pieces + c];
        Vc[(size_t)row * pieces + cd] = vs[(size_t)r * pieces + c];
    }
    if (blockIdx.x != 0) return;
    for (int a = threadIdx.x; a < W + R; a += blockDim.x) {
        float zz = -INFINITY;
        if (a < W) {
            // slot a holds the newest position congruent to a (mod W), if there is one yet
            const int lo = n1 - Wnew;
            const int pos = lo + ((a - lo % W) + W) % W;
            if (pos < n1 && pos <= n1 - 1 - half) zz = zl[Tloc - (n1 - pos)];
        } else if (a - W < cnt) {
            const int r = idx[(size_t)bh * R + (a - W)];
            zz = zl[r];
            pidx[a - W] = r < R0 ? oldpos[(size_t)bh * R + r] : n0 - Wn + (r - R0);
        }
        zc[a] = zz;
    }
    if (threadIdx.x == 0) { meta[0] = n1; meta[1] = cnt; }
}

// The streaming reading (Section 3.1.3, decoding paragraph, applied inside a chunk): one warp per (b,h) walks the chunk's
// queries in order and applies the replace-the-lowest rule to the token each query pushes out of its window (local row
// rq - W).  Out: the list of every entry that is in the pool at some query of the chunk (local rows, in order of
// entering = ascending; the pool the cache held comes first), for each the query row from which it is gone (`leave`,
// INT_MAX for the survivors), and the survivors as the new pool (idx, cnt; ascending local rows).  zrank holds the logits
// of the local sequence with sink tokens at +inf; keep iff zrank > zthr.
__global__ void __launch_bounds__(32) chunk_stream_kernel(const float* __restrict__ zrank, const int32_t* __restrict__ oldpos,
                                                          int32_t* __restrict__ ulist, int32_t* __restrict__ leave,
                                                          int32_t* __restrict__ ucnt, int32_t* __restrict__ idx,
                                                          int32_t* __restrict__ cnt, int R, int W, int Tloc, int ucap, int n0,
                                                          int R0, int Wn, float zthr)
{
    extern __shared__ int sm_i[];
    float* pz = reinterpret_cast<float*>(sm_i);                // [R] logit of pool entry
    int* ppos = sm_i + R;                                       // [R] position (for the tie rule: the youngest of equals goes)
    int* pu = sm_i + 2 * R;                                     // [R] its index in the entry list
    const int bh = blockIdx.x, lane = threadIdx.x;
    const float* zr = zrank + (size_t)bh * Tloc;
    const int32_t* op = oldpos + (size_t)bh * R;
    int32_t* ul = ulist + (size_t)bh * ucap;
    int32_t* lv = leave + (size_t)bh * ucap;
    int n_pool = 0;
    if (R0 > 0) {                                              // the pool the cache holds: local rows [0, its count)
        for (int e = lane; e < R; e += 32) {
            const bool ok = op[e] >= 0;
            if (ok) { pz[e] = zr[e]; ppos[e] = op[e]; pu[e] = e; ul[e] = e; lv[e] = 0x7fffffff; }
            n_pool += ok ? 1 : 0;                              // valid slots are the first ones
        }
        n_pool = __reduce_add_sync(0xffffffffu, n_pool);
    }
    int n_u = n_pool;
    __syncwarp();
    const int Tc = Tloc - R0 - Wn;
    // The lowest entry of a full pool only ever rises (a replacement puts a higher logit in its place), so a token at or
    // below it can be dropped without looking at the pool again: the lowest entry is searched once after every
    // replacement, and 32 tokens at a time are tested against it with one ballot.
    bool worst_known = false;
    float wz = INFINITY; int wp = -1, wi = -1;
    auto find_worst = [&]() {                                  // the lowest logit; among equals the youngest
        wz = INFINITY; wp = -1; wi = -1;
        for (int e = lane; e < R; e += 32) {
            const float ze = pz[e]; const int pe = ppos[e];
            if (ze < wz || (ze == wz && pe > wp)) { wz = ze; wp = pe; wi = e; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float oz = __shfl_xor_sync(0xffffffffu, wz, o);
            const int opp = __shfl_xor_sync(0xffffffffu, wp, o), oi = __shfl_xor_sync(0xffffffffu, wi, o);
            if (oz < wz || (oz == wz && opp > wp)) { wz = oz; wp = opp; wi = oi; }
        }
        worst_known = true;
    };
    for (int t0 = 0; t0 < Tc && R > 0; t0 += 32) {
        // lane l: the token that query t0 + l pushes out of its window (local row rq - W), if it passes the threshold
        const int my_rq = R0 + Wn + t0 + lane, my_r = my_rq - W;
        const float my_z = (t0 + lane < Tc && my_r >= R0) ? zr[my_r] : -INFINITY;
        unsigned todo = __ballot_sync(0xffffffffu, my_z > zthr);
        if (worst_known) todo &= __ballot_sync(0xffffffffu, my_z > wz);
        while (todo != 0u) {
            const int l = __ffs(todo) - 1;
            todo &= todo - 1u;
            const float zc = __shfl_sync(0xffffffffu, my_z, l);
            const int rq = R0 + Wn + t0 + l, r = rq - W;
            const int pos = n0 - Wn + (r - R0);
            if (n_pool < R) {
                if (lane == 0) { pz[n_pool] = zc; ppos[n_pool] = pos; pu[n_pool] = n_u; ul[n_u] = r; lv[n_u] = 0x7fffffff; }
                ++n_pool; ++n_u;
                __syncwarp();
                continue;
            }
            if (!worst_known) find_worst();
            if (wi >= 0 && zc > wz) {                            // strictly better: the entry is gone from this query on
                if (lane == 0) { lv[pu[wi]] = rq; pz[wi] = zc; ppos[wi] = pos; pu[wi] = n_u; ul[n_u] = r; lv[n_u] = 0x7fffffff; }
                ++n_u;
                __syncwarp();
                find_worst();
            }
            todo &= __ballot_sync(0xffffffffu, my_z > wz);      // the later tokens of the batch against the new lowest entry
        }
    }
    __syncwarp();
    // the survivors, in list order (ascending local rows), are the new pool
    int n_out = 0;
    for (int e0 = 0; e0 < n_u; e0 += 32) {
        const int e = e0 + lane;
        const bool keep = e < n_u && lv[e] == 0x7fffffff;
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
        if (keep) idx[(size_t)bh * R + n_out + __popc(bal & ((1u << lane) - 1u))] = ul[e];
        n_out += __popc(bal);
    }
    for (int e = n_out + lane; e < R; e += 32) idx[(size_t)bh * R + e] = -1;
    if (lane == 0) { cnt[bh] = n_out; ucnt[bh] = n_u; }
}

}  // namespace

int launch_chunk_stream(const Params& p, const float* zrank, const int32_t* oldpos, int32_t* ulist, int32_t* leave, int32_t* ucnt,
                        int32_t* idx, int32_t* cnt, int ucap, int n0, int R0, int Wn, cudaStream_t st)
{
    const size_t smem = (size_t)(p.R > 0 ? p.R : 1) * 12;
    if (smem > 48 * 1024) return LTE_ERR_UNSUPPORTED;           // pools of up to 4096 entries
    chunk_stream_kernel<<<p.B * p.H, 32, smem, st>>>(zrank, oldpos, ulist, leave, ucnt, idx, cnt, p.R, p.W, p.T, ucap, n0, R0, Wn, p.zthr);
    return cuda_status(cudaGetLastError());
}

int chunk_status_fetch_and_clear() { return status_fetch_and_clear(g_chunk_status); }

// p.T = local length; the launchers run on one stream in the order gather, (scores), merge, (select, attention), commit
int launch_chunk_gather(const Params& p, const void* cache, const void* k, const void* v, void* klin, void* vlin, float* zsrc,
                        int32_t* oldpos, int32_t* gate, int n0, int R0, int Wn, cudaStream_t st)
{
    const CacheLayout L = cache_layout(p.d, p.W, p.R, p.dtype);
    dim3 grid((p.T + kRowsPerBlock - 1) / kRowsPerBlock, p.B * p.H);
    chunk_gather_kernel<<<grid, 256, 0, st>>>((const unsigned char*)cache, L, (const unsigned char*)k, (const unsigned char*)v,
                                              (unsigned char*)klin, (unsigned char*)vlin, zsrc, oldpos, gate, p.d, p.W, p.R, n0, R0, Wn, p.T);
    return cuda_status(cudaGetLastError());
}

int launch_chunk_merge_z(const Params& p, float* z, float* zrank, const float* zsrc, const int32_t* oldpos, int n0, int R0, int Wn,
                         cudaStream_t st)
{
    dim3 grid((p.T + 255) / 256, p.B * p.H);
    chunk_merge_z_kernel<<<grid, 256, 0, st>>>(z, zrank, zsrc, oldpos, p.R, p.W, n0, R0, Wn, p.T, p.half, p.sink);
    return cuda_status(cudaGetLastError());
}

int launch_chunk_commit(const Params& p, void* cache, const void* klin, const void* vlin, const float* z, const int32_t* idx,
                        const int32_t* cnt, const int32_t* oldpos, const int32_t* gate, int n0, int n1, int R0, int Wn,
                        cudaStream_t st)
{
    const CacheLayout L = cache_layout(p.d, p.W, p.R, p.dtype);
    dim3 grid((p.W + p.R + kRowsPerBlock - 1) / kRowsPerBlock, p.B * p.H);
    chunk_commit_kernel<<<grid, 256, 0, st>>>((unsigned char*)cache, L, (const unsigned char*)klin, (const unsigned char*)vlin, z,
                                                   idx, cnt, oldpos, gate, p.d, p.W, p.R, n0, n1, R0, Wn, p.T, p.half);
    return cuda_status(cudaGetLastError());
}

}  // namespace lte
