// Backward of the paper's scorer stack (Section 3.1.1's module under the gradient of Section 3.1.2), d = 64, fp32 on
// the ordinary ALUs: given dL/dz per token (the straight-through surrogate has already produced it), the gradients of
// the three conv layers' weights and biases and of the output map, and optionally the gradient into k and v.
//
// A CTA keeps one head's weights in shared memory ([tap][c_in][c_out + 4], the layout both the forward products and
// the transposed ones read without bank conflicts) and walks tiles of 32 times [a, a+32) of one (b,h) row:
//   forward again over the rows the tile's gradients reach (inputs a-12 .. a+43, then h0, h1, h2 on shrinking ranges),
//   keeping every layer's activation and Swish'(y);
//   delta2 = dz wout Swish'(y2), then per layer, going down: the weight gradient sum_{t in tile} delta_l[t] x in_l[t - shift]
//   accumulated in registers across the CTA's tiles, and delta_{l-1}[t'] = Swish'(y_{l-1}[t']) sum_tau W_l[tau]^T delta_l[t' + shift]
//   written over the Swish' buffer it multiplies; the last one is the input gradient, added to dk, dv.
// Each time is owned by one tile (gradients outside [0, T) are zero by construction), so the per-CTA partial sums,
// written to scratch at the end, add up to the full gradients in a second, fixed-order kernel: deterministic.
#include "common.cuh"

namespace lte {
namespace {

constexpr int SB_NT = 256, SB_TR = 32;
constexpr int SB_C0 = 128, SB_C1 = 64, SB_C2 = 32, SB_C3 = 16;
// rows of a tile: x from a-12, h0 from a-8, h1 from a-4, h2 from a; all end at a + TR + 12
constexpr int SB_RX = SB_TR + 24, SB_R0 = SB_TR + 20, SB_R1 = SB_TR + 16, SB_R2 = SB_TR + 12;
constexpr int SB_SX = SB_C0 + 4, SB_S0 = SB_C1 + 4, SB_S1 = SB_C2 + 4, SB_S2 = SB_C3 + 4;   // row strides (floats)
constexpr int SB_W0 = 3 * SB_C0 * (SB_C1 + 4), SB_W1 = 3 * SB_C1 * (SB_C2 + 4), SB_W2 = 3 * SB_C2 * (SB_C3 + 4);
constexpr int SB_OFF_W0 = 0, SB_OFF_W1 = SB_OFF_W0 + SB_W0, SB_OFF_W2 = SB_OFF_W1 + SB_W1, SB_OFF_P = SB_OFF_W2 + SB_W2;
constexpr int SB_OFF_X = SB_OFF_P + 144;                       // parameters: b0[64] b1[32] b2[16] wout[16] bout
constexpr int SB_OFF_H0 = SB_OFF_X + SB_RX * SB_SX, SB_OFF_D0 = SB_OFF_H0 + SB_R0 * SB_S0;
constexpr int SB_OFF_H1 = SB_OFF_D0 + SB_R0 * SB_S0, SB_OFF_D1 = SB_OFF_H1 + SB_R1 * SB_S1;
constexpr int SB_OFF_H2 = SB_OFF_D1 + SB_R1 * SB_S1, SB_OFF_D2 = SB_OFF_H2 + SB_R2 * SB_S2;
constexpr int SB_OFF_DZ = SB_OFF_D2 + SB_R2 * SB_S2;           // delta3 of the tile's rows [SB_R2]
constexpr int SB_FLOATS = SB_OFF_DZ + ((SB_R2 + 3) & ~3);
constexpr size_t SB_BYTES = (size_t)SB_FLOATS * sizeof(float);
static_assert(SB_BYTES <= 232448, "shared memory");
// packed gradient layout of one head (floats): wl0 [64][3][128] | wl1 [32][3][64] | wl2 [16][3][32] | wout [16] | b0 | b1 | b2 | bout
constexpr int SB_G0 = SB_C1 * 3 * SB_C0, SB_G1 = SB_C2 * 3 * SB_C1, SB_G2 = SB_C3 * 3 * SB_C2;
constexpr int SB_PART = SB_G0 + SB_G1 + SB_G2 + SB_C3 + SB_C1 + SB_C2 + SB_C3 + 1;   // 32,385
constexpr int SB_PART_PAD = (SB_PART + 31) & ~31;

// Forward layer: out[r][o] = Swish(y), sp[r][o] = Swish'(y), y = bias[o] + sum_{tau, c} w[tau][c][o] in[r + 2 tau][c];
// out row r is at time t_out0 + r (zero, with zero derivative, at negative times); in row 0 is at time t_out0 - 4.
template <int CIN, int COUT, int ROWS, int SIN, int SOUT>
__device__ __forceinline__ void sb_forward(const float* __restrict__ in, float* __restrict__ out, float* __restrict__ sp,
                                           const float* __restrict__ w, const float* __restrict__ bias, int t_out0)
{
    constexpr int TX = COUT / 4, TY = SB_NT / TX, RPT = (ROWS + TY - 1) / TY, WS = COUT + 4;
    const int tx = threadIdx.x % TX, ty = threadIdx.x / TX;
    float acc[RPT][4];
    int rrow[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        rrow[i] = min(ty + TY * i, ROWS - 1);                  // surplus threads recompute the last row
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
    }
#pragma unroll 1
    for (int tau = 0; tau < 3; ++tau) {
#pragma unroll 2
        for (int c = 0; c < CIN; c += 4) {
            float4 a[RPT];
#pragma unroll
            for (int i = 0; i < RPT; ++i) a[i] = *reinterpret_cast<const float4*>(&in[(rrow[i] + 2 * tau) * SIN + c]);
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const float4 b = *reinterpret_cast<const float4*>(&w[(tau * CIN + c + cc) * WS + 4 * tx]);
#pragma unroll
                for (int i = 0; i < RPT; ++i) {
                    const float av = cc == 0 ? a[i].x : cc == 1 ? a[i].y : cc == 2 ? a[i].z : a[i].w;
                    acc[i][0] = fmaf(av, b.x, acc[i][0]); acc[i][1] = fmaf(av, b.y, acc[i][1]);
                    acc[i][2] = fmaf(av, b.z, acc[i][2]); acc[i][3] = fmaf(av, b.w, acc[i][3]);
                }
            }
        }
    }
    const float4 bb = *reinterpret_cast<const float4*>(&bias[4 * tx]);
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const int r = ty + TY * i;
        if (r < ROWS) {
            const float live = t_out0 + r >= 0 ? 1.f : 0.f;
            const float y[4] = {acc[i][0] + bb.x, acc[i][1] + bb.y, acc[i][2] + bb.z, acc[i][3] + bb.w};
            float h[4], s[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float sg = 1.f / (1.f + expf(-y[e]));
                h[e] = live * y[e] * sg;
                s[e] = live * sg * (1.f + y[e] * (1.f - sg));
            }
            *reinterpret_cast<float4*>(&out[r * SOUT + 4 * tx]) = make_float4(h[0], h[1], h[2], h[3]);
            *reinterpret_cast<float4*>(&sp[r * SOUT + 4 * tx]) = make_float4(s[0], s[1], s[2], s[3]);
        }
    }
}

// Transposed layer: g[r][c] = sum_{tau', o} delta[r + 2 tau'][o] w[2 - tau'][c][o] for rows r < ROWS (delta row 0 and
// g row 0 at the same time); a thread owns channels tx, tx + TX, tx + 2 TX, tx + 3 TX (consecutive threads read
// consecutive weight rows: conflict-free 16-byte loads along o).  fn(r, c, g) receives every result.
template <int CO, int CI, int ROWS, int SD, typename F>
__device__ __forceinline__ void sb_transposed(const float* __restrict__ delta, const float* __restrict__ w, F fn)
{
    constexpr int TX = CI / 4, TY = SB_NT / TX, RPT = (ROWS + TY - 1) / TY, WS = CO + 4;
    const int tx = threadIdx.x % TX, ty = threadIdx.x / TX;
    float acc[RPT][4];
    int rrow[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        rrow[i] = min(ty + TY * i, ROWS - 1);
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
    }
#pragma unroll 1
    for (int tp = 0; tp < 3; ++tp) {
        const int tau = 2 - tp;
#pragma unroll 2
        for (int o = 0; o < CO; o += 4) {
            float4 wv[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) wv[j] = *reinterpret_cast<const float4*>(&w[(tau * CI + tx + j * TX) * WS + o]);
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                const float4 d4 = *reinterpret_cast<const float4*>(&delta[(rrow[i] + 2 * tp) * SD + o]);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    acc[i][j] = fmaf(d4.x, wv[j].x, fmaf(d4.y, wv[j].y, fmaf(d4.z, wv[j].z, fmaf(d4.w, wv[j].w, acc[i][j]))));
            }
        }
    }
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const int r = ty + TY * i;
        if (r < ROWS)
#pragma unroll
            for (int j = 0; j < 4; ++j) fn(r, tx + j * TX, acc[i][j]);
    }
}

// Weight gradient of one layer over the tile's own times: acc[tau][j][cc] += delta[t][4 ob + j] in[t + 2 tau][cb CB + cc],
// t < SB_TR.  delta row 0 is time a; in row 0 is time a - 4.  Threads beyond CO/4 * CI/CB take no part.
template <int CO, int CI, int CB, int SD, int SIN>
__device__ __forceinline__ void sb_wgrad(float (&acc)[3][4][CB], const float* __restrict__ delta, const float* __restrict__ in)
{
    constexpr int NCB = CI / CB;
    if (threadIdx.x >= (CO / 4) * NCB) return;
    const int cb = threadIdx.x % NCB, ob = threadIdx.x / NCB;
#pragma unroll 2
    for (int t = 0; t < SB_TR; ++t) {
        const float4 d4 = *reinterpret_cast<const float4*>(&delta[t * SD + 4 * ob]);
        const float dv[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
        for (int tau = 0; tau < 3; ++tau) {
            float xv[CB];
            if constexpr (CB % 4 == 0) {
#pragma unroll
                for (int cc = 0; cc < CB; cc += 4) {
                    const float4 x4 = *reinterpret_cast<const float4*>(&in[(t + 2 * tau) * SIN + cb * CB + cc]);
                    xv[cc] = x4.x; xv[cc + 1] = x4.y; xv[cc + 2] = x4.z; xv[cc + 3] = x4.w;
                }
            } else {
#pragma unroll
                for (int cc = 0; cc < CB; ++cc) xv[cc] = in[(t + 2 * tau) * SIN + cb * CB + cc];
            }
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int cc = 0; cc < CB; ++cc) acc[tau][j][cc] = fmaf(dv[j], xv[cc], acc[tau][j][cc]);
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(SB_NT, 1)
stack_bwd_kernel(const T* __restrict__ k, const T* __restrict__ v, const float* __restrict__ wpack,
                 const float* __restrict__ bpack, const float* __restrict__ dz, T* __restrict__ dk, T* __restrict__ dv,
                 float* __restrict__ part, int H, int Tlen, int tiles_per_cta, int input_grad)
{
    extern __shared__ __align__(16) float sm[];
    pdl_launch_dependents();
    pdl_wait();
    constexpr int D = 64;
    const int bh = blockIdx.y, h = bh % H, tid = threadIdx.x;
    const int n_tiles = (Tlen + SB_TR - 1) / SB_TR;
    const int tile_begin = blockIdx.x * tiles_per_cta, tile_end = min(tile_begin + tiles_per_cta, n_tiles);
    float* my_part = part + ((size_t)bh * gridDim.x + blockIdx.x) * SB_PART_PAD;

    // ---- this head's parameters: weights as [tap][c_in][c_out + 4] ----
    const float* g0 = wpack + (size_t)h * SB_G0;
    const float* g1 = wpack + (size_t)H * SB_G0 + (size_t)h * SB_G1;
    const float* g2 = wpack + (size_t)H * (SB_G0 + SB_G1) + (size_t)h * SB_G2;
    const float* go = wpack + (size_t)H * (SB_G0 + SB_G1 + SB_G2) + (size_t)h * SB_C3;
    for (int e = tid; e < SB_G0; e += SB_NT) {                 // e = (o * 3 + tau) * C0 + c
        const int c = e % SB_C0, ot = e / SB_C0, tau = ot % 3, o = ot / 3;
        sm[SB_OFF_W0 + (tau * SB_C0 + c) * (SB_C1 + 4) + o] = g0[e];
    }
    for (int e = tid; e < SB_G1; e += SB_NT) {
        const int c = e % SB_C1, ot = e / SB_C1, tau = ot % 3, o = ot / 3;
        sm[SB_OFF_W1 + (tau * SB_C1 + c) * (SB_C2 + 4) + o] = g1[e];
    }
    for (int e = tid; e < SB_G2; e += SB_NT) {
        const int c = e % SB_C2, ot = e / SB_C2, tau = ot % 3, o = ot / 3;
        sm[SB_OFF_W2 + (tau * SB_C2 + c) * (SB_C3 + 4) + o] = g2[e];
    }
    for (int e = tid; e < 144; e += SB_NT) {
        float b = 0.f;
        if (e < 64) b = bpack ? bpack[(size_t)h * 64 + e] : 0.f;
        else if (e < 96) b = bpack ? bpack[(size_t)H * 64 + (size_t)h * 32 + (e - 64)] : 0.f;
        else if (e < 112) b = bpack ? bpack[(size_t)H * 96 + (size_t)h * 16 + (e - 96)] : 0.f;
        else if (e < 128) b = go[e - 112];
        else if (e == 128) b = bpack ? bpack[(size_t)H * 112 + h] : 0.f;
        sm[SB_OFF_P + e] = b;
    }
    const float* sb0 = sm + SB_OFF_P, *sb1 = sm + SB_OFF_P + 64, *sb2 = sm + SB_OFF_P + 96, *swo = sm + SB_OFF_P + 112;

    // gradient accumulators of this CTA (registers, across its tiles)
    float a0[3][4][8], a1[3][4][2], a2[3][4][1];
#pragma unroll
    for (int t = 0; t < 3; ++t)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
            for (int c = 0; c < 8; ++c) a0[t][j][c] = 0.f;
            a1[t][j][0] = a1[t][j][1] = 0.f;
            a2[t][j][0] = 0.f;
        }
    float small = 0.f;                                         // thread < 64: db0; < 96: db1; < 112: db2; < 128: dwout; 128: dbout

    const T* kk = k + (size_t)bh * Tlen * D;
    const T* vv = v + (size_t)bh * Tlen * D;
    const float* dzz = dz + (size_t)bh * Tlen;
    for (int tile = tile_begin; tile < tile_end; ++tile) {
        const int a = tile * SB_TR;                            // the tile owns times a .. a + TR - 1
        __syncthreads();                                       // the previous tile's readers are done (and the parameters are in)
        // ---- input rows a-12 .. a+TR+11 (zero outside [0, T)) and delta3[t] = dz[t - 6] for the rows a .. a+TR+11 ----
        for (int e = tid; e < SB_RX * (SB_C0 / 4); e += SB_NT) {
            const int r = e / (SB_C0 / 4), c4 = (e % (SB_C0 / 4)) * 4;
            const int t = a - 12 + r;
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (t >= 0 && t < Tlen) {
                const T* src = (c4 < D ? kk : vv) + (size_t)t * D + (c4 < D ? c4 : c4 - D);
                if constexpr (sizeof(T) == 2) {
                    const uint2 u = *reinterpret_cast<const uint2*>(src);
                    x = make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u),
                                    __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
                } else {
                    x = *reinterpret_cast<const float4*>(src);
                }
            }
            *reinterpret_cast<float4*>(&sm[SB_OFF_X + r * SB_SX + c4]) = x;
        }
        if (tid < SB_R2) {
            const int t = a + tid;
            sm[SB_OFF_DZ + tid] = (t >= 6 && t < Tlen) ? dzz[t - 6] : 0.f;   // the caller's dz is zero where the logit is undefined
        }
        __syncthreads();
        // ---- forward, keeping activations and Swish' ----
        sb_forward<SB_C0, SB_C1, SB_R0, SB_SX, SB_S0>(sm + SB_OFF_X, sm + SB_OFF_H0, sm + SB_OFF_D0, sm + SB_OFF_W0, sb0, a - 8);
        __syncthreads();
        sb_forward<SB_C1, SB_C2, SB_R1, SB_S0, SB_S1>(sm + SB_OFF_H0, sm + SB_OFF_H1, sm + SB_OFF_D1, sm + SB_OFF_W1, sb1, a - 4);
        __syncthreads();
        sb_forward<SB_C2, SB_C3, SB_R2, SB_S1, SB_S2>(sm + SB_OFF_H1, sm + SB_OFF_H2, sm + SB_OFF_D2, sm + SB_OFF_W2, sb2, a);
        __syncthreads();
        // ---- output map: dwout, dbout over the tile's own times; delta2 = delta3 wout Swish'(y2) in place ----
        if (tid >= 112 && tid <= 128) {
            for (int t = 0; t < SB_TR; ++t) {
                const float d3 = sm[SB_OFF_DZ + t];
                small += tid == 128 ? d3 : d3 * sm[SB_OFF_H2 + t * SB_S2 + (tid - 112)];
            }
        }
        __syncthreads();
        for (int e = tid; e < SB_R2 * SB_C3; e += SB_NT) {
            const int r = e / SB_C3, c = e % SB_C3;
            sm[SB_OFF_D2 + r * SB_S2 + c] *= sm[SB_OFF_DZ + r] * swo[c];
        }
        __syncthreads();
        // ---- layer 2: weight gradient (delta2 x h1), bias, then delta1 into the Swish' buffer of layer 1 (rows from a) ----
        sb_wgrad<SB_C3, SB_C2, 1, SB_S2, SB_S1>(a2, sm + SB_OFF_D2, sm + SB_OFF_H1);
        if (tid >= 96 && tid < 112)
            for (int t = 0; t < SB_TR; ++t) small += sm[SB_OFF_D2 + t * SB_S2 + (tid - 96)];
        sb_transposed<SB_C3, SB_C2, SB_TR + 8, SB_S2>(sm + SB_OFF_D2, sm + SB_OFF_W2,
                                                      [&](int r, int c, float g) { sm[SB_OFF_D1 + (r + 4) * SB_S1 + c] *= g; });
        __syncthreads();
        // ---- layer 1 ----
        sb_wgrad<SB_C2, SB_C1, 2, SB_S1, SB_S0>(a1, sm + SB_OFF_D1 + 4 * SB_S1, sm + SB_OFF_H0 + 4 * SB_S0);
        if (tid >= 64 && tid < 96)
            for (int t = 0; t < SB_TR; ++t) small += sm[SB_OFF_D1 + (t + 4) * SB_S1 + (tid - 64)];
        sb_transposed<SB_C2, SB_C1, SB_TR + 4, SB_S1>(sm + SB_OFF_D1 + 4 * SB_S1, sm + SB_OFF_W1,
                                                      [&](int r, int c, float g) { sm[SB_OFF_D0 + (r + 8) * SB_S0 + c] *= g; });
        __syncthreads();
        // ---- layer 0 ----
        sb_wgrad<SB_C1, SB_C0, 8, SB_S0, SB_SX>(a0, sm + SB_OFF_D0 + 8 * SB_S0, sm + SB_OFF_X + 8 * SB_SX);
        if (tid < 64)
            for (int t = 0; t < SB_TR; ++t) small += sm[SB_OFF_D0 + (t + 8) * SB_S0 + tid];
        if (input_grad) {
            // the gradient into the inputs: channels [0, 64) into dk, [64, 128) into dv, added to what the attention left there
            sb_transposed<SB_C1, SB_C0, SB_TR, SB_S0>(sm + SB_OFF_D0 + 8 * SB_S0, sm + SB_OFF_W0, [&](int r, int c, float g) {
                const int t = a + r;
                if (t < Tlen) {
                    T* dst = (c < D ? dk : dv) + ((size_t)bh * Tlen + t) * D + (c < D ? c : c - D);
                    *dst = from_f<T>(to_f(*dst) + g);
                }
            });
        }
    }
    // ---- this CTA's partial sums, in the packed layout of the parameters ----
    {
        const int cb = tid % 16, ob = tid / 16;                // layer 0: 16 blocks of 4 outputs x 16 blocks of 8 inputs
#pragma unroll
        for (int tau = 0; tau < 3; ++tau)
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int cc = 0; cc < 8; ++cc) my_part[((4 * ob + j) * 3 + tau) * SB_C0 + cb * 8 + cc] = a0[tau][j][cc];
    }
    {
        const int cb = tid % 32, ob = tid / 32;                // layer 1: 8 x 32 blocks of 4 x 2
#pragma unroll
        for (int tau = 0; tau < 3; ++tau)
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) my_part[SB_G0 + ((4 * ob + j) * 3 + tau) * SB_C1 + cb * 2 + cc] = a1[tau][j][cc];
    }
    if (tid < 128) {
        const int cb = tid % 32, ob = tid / 32;                // layer 2: 4 x 32 blocks of 4 x 1
#pragma unroll
        for (int tau = 0; tau < 3; ++tau)
#pragma unroll
            for (int j = 0; j < 4; ++j) my_part[SB_G0 + SB_G1 + ((4 * ob + j) * 3 + tau) * SB_C2 + cb] = a2[tau][j][0];
    }
    {
        // wout [16] | b0 [64] | b1 [32] | b2 [16] | bout
        float* sp = my_part + SB_G0 + SB_G1 + SB_G2;
        if (tid < 64) sp[16 + tid] = small;
        else if (tid < 96) sp[16 + 64 + (tid - 64)] = small;
        else if (tid < 112) sp[16 + 96 + (tid - 96)] = small;
        else if (tid < 128) sp[tid - 112] = small;
        else if (tid == 128) sp[16 + 112] = small;
    }
}

// dw = wl0 | wl1 | wl2 | wout (every tensor over all heads), dbias = bl0 | bl1 | bl2 | bout: sums of the partials of a head's
// CTAs (all batch elements, all row chunks) in a fixed order.
__global__ void stack_bwd_reduce_kernel(const float* __restrict__ part, float* __restrict__ dw, float* __restrict__ dbias,
                                        int B, int H, int chunks)
{
    pdl_launch_dependents();
    pdl_wait();
    const int h = blockIdx.y, e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= SB_PART) return;
    float t = 0.f;
    for (int b = 0; b < B; ++b)
        for (int ch = 0; ch < chunks; ++ch) t += part[(((size_t)b * H + h) * chunks + ch) * SB_PART_PAD + e];
    if (e < SB_G0) dw[(size_t)h * SB_G0 + e] = t;
    else if (e < SB_G0 + SB_G1) dw[(size_t)H * SB_G0 + (size_t)h * SB_G1 + (e - SB_G0)] = t;
    else if (e < SB_G0 + SB_G1 + SB_G2) dw[(size_t)H * (SB_G0 + SB_G1) + (size_t)h * SB_G2 + (e - SB_G0 - SB_G1)] = t;
    else if (e < SB_G0 + SB_G1 + SB_G2 + 16) dw[(size_t)H * (SB_G0 + SB_G1 + SB_G2) + (size_t)h * 16 + (e - SB_G0 - SB_G1 - SB_G2)] = t;
    else if (dbias) {
        const int f = e - (SB_G0 + SB_G1 + SB_G2 + 16);        // b0 [64] | b1 [32] | b2 [16] | bout
        if (f < 64) dbias[(size_t)h * 64 + f] = t;
        else if (f < 96) dbias[(size_t)H * 64 + (size_t)h * 32 + (f - 64)] = t;
        else if (f < 112) dbias[(size_t)H * 96 + (size_t)h * 16 + (f - 96)] = t;
        else dbias[(size_t)H * 112 + h] = t;
    }
}

int stack_bwd_chunks(const Params& p)
{
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int BH = p.B * p.H, n_tiles = (p.T + SB_TR - 1) / SB_TR;
    int chunks = (2 * sms + BH - 1) / BH;                      // about two waves of CTAs: the tail of the last wave stays short
    if (chunks < 1) chunks = 1;
    if (chunks > n_tiles) chunks = n_tiles;
    const int per = (n_tiles + chunks - 1) / chunks;
    return (n_tiles + per - 1) / per;
}

}  // namespace

// Scratch of the stack's backward: one packed partial gradient per CTA.
size_t stack_bwd_workspace(const Params& p)
{
    if (p.d != 64) return 0;
    return (size_t)p.B * p.H * stack_bwd_chunks(p) * SB_PART_PAD * sizeof(float);
}

// dz [B,H,T] fp32 (zero where the logit is undefined) -> dw, dbias (packed like the parameters; dbias may be null) and,
// with input_grad, dk += , dv += the gradient into the scorer's inputs.  part: stack_bwd_workspace(p) bytes.
int launch_stack_bwd(const Params& p, const void* k, const void* v, const float* dz, void* dk, void* dv, float* dw,
                     float* dbias, bool input_grad, void* part, cudaStream_t st)
{
    if (p.d != 64) return LTE_ERR_UNSUPPORTED;
    const int chunks = stack_bwd_chunks(p);
    const int n_tiles = (p.T + SB_TR - 1) / SB_TR, per = (n_tiles + chunks - 1) / chunks;
    dim3 grid(chunks, p.B * p.H);
    cudaError_t e;
    if (p.dtype == LTE_BF16) {
        static PerDeviceOnce attr;
        if (int e2 = attr.run([] { return cudaFuncSetAttribute(stack_bwd_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SB_BYTES); }))
            return e2;
        e = launch_pdl(stack_bwd_kernel<__nv_bfloat16>, grid, dim3(SB_NT), SB_BYTES, st, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v,
                       p.w, p.bias, dz, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, (float*)part, p.H, p.T, per, input_grad ? 1 : 0);
    } else {
        static PerDeviceOnce attr;
        if (int e2 = attr.run([] { return cudaFuncSetAttribute(stack_bwd_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SB_BYTES); }))
            return e2;
        e = launch_pdl(stack_bwd_kernel<float>, grid, dim3(SB_NT), SB_BYTES, st, (const float*)k, (const float*)v, p.w, p.bias, dz,
                       (float*)dk, (float*)dv, (float*)part, p.H, p.T, per, input_grad ? 1 : 0);
    }
    if (e != cudaSuccess) return LTE_ERR_CUDA;
    if (launch_pdl(stack_bwd_reduce_kernel, dim3((SB_PART + 255) / 256, p.H), dim3(256), 0, st, (const float*)part, dw, dbias, p.B,
                   p.H, chunks) != cudaSuccess)
        return LTE_ERR_CUDA;
    return cuda_status(cudaGetLastError());
}

}  // namespace lte
