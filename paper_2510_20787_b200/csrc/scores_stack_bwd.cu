// Backward of the paper's scorer stack (Section 3.1.1's module under the gradient of Section 3.1.2), d = 64 or 32, fp32 on
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
// rows of a tile: x from a-12, h0 from a-8, h1 from a-4, h2 from a; all end at a + TR + 12
constexpr int SB_RX = SB_TR + 24, SB_R0 = SB_TR + 20, SB_R1 = SB_TR + 16, SB_R2 = SB_TR + 12;
// Channel plan 2d -> d -> d/2 -> d/4 -> 1 and everything that follows from it (d = 64 or 32).
template <int D> struct SBL {
    static constexpr int C0 = 2 * D, C1 = D, C2 = D / 2, C3 = D / 4;
    static constexpr int SX = C0 + 4, S0 = C1 + 4, S1 = C2 + 4, S2 = C3 + 4;   // row strides (floats)
    static constexpr int W0 = 3 * C0 * (C1 + 4), W1 = 3 * C1 * (C2 + 4), W2 = 3 * C2 * (C3 + 4);
    static constexpr int OFF_W0 = 0, OFF_W1 = OFF_W0 + W0, OFF_W2 = OFF_W1 + W1, OFF_P = OFF_W2 + W2;
    // parameters: b0[C1] b1[C2] b2[C3] wout[C3] bout; the same thread numbers own their gradients
    static constexpr int P1 = C1, P2 = P1 + C2, P3 = P2 + C3, P4 = P3 + C3, NP = P4 + 1, NP_PAD = (NP + 15) & ~15;
    static constexpr int OFF_X = OFF_P + NP_PAD;
    static constexpr int OFF_H0 = OFF_X + SB_RX * SX, OFF_D0 = OFF_H0 + SB_R0 * S0;
    static constexpr int OFF_H1 = OFF_D0 + SB_R0 * S0, OFF_D1 = OFF_H1 + SB_R1 * S1;
    static constexpr int OFF_H2 = OFF_D1 + SB_R1 * S1, OFF_D2 = OFF_H2 + SB_R2 * S2;
    static constexpr int OFF_DZ = OFF_D2 + SB_R2 * S2;         // delta3 of the tile's rows [SB_R2]
    static constexpr int FLOATS = OFF_DZ + ((SB_R2 + 3) & ~3);
    static constexpr size_t BYTES = (size_t)FLOATS * sizeof(float);
    static_assert(BYTES <= 232448, "shared memory");
    // packed gradient layout of one head (floats): wl0 [C1][3][C0] | wl1 [C2][3][C1] | wl2 [C3][3][C2] | wout [C3] | b0 | b1 | b2 | bout
    static constexpr int G0 = C1 * 3 * C0, G1 = C2 * 3 * C1, G2 = C3 * 3 * C2;
    static constexpr int PART = G0 + G1 + G2 + C3 + C1 + C2 + C3 + 1;   // 32,385 at d = 64
    static constexpr int PART_PAD = (PART + 31) & ~31;
    // input channels per thread in the weight-gradient products (a thread owns 4 outputs x CB inputs x 3 taps)
    static constexpr int CB0 = D == 64 ? 8 : 2, CB1 = D == 64 ? 2 : 1, CB2 = 1;
    static_assert((C1 / 4) * (C0 / CB0) <= SB_NT && (C2 / 4) * (C1 / CB1) <= SB_NT && (C3 / 4) * (C2 / CB2) <= SB_NT, "threads");
};

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

template <typename T, int D>
__global__ void __launch_bounds__(SB_NT, 1)
stack_bwd_kernel(const T* __restrict__ k, const T* __restrict__ v, const float* __restrict__ wpack,
                 const float* __restrict__ bpack, const float* __restrict__ dz, T* __restrict__ dk, T* __restrict__ dv,
                 float* __restrict__ part, int H, int Tlen, int tiles_per_cta, int input_grad)
{
    extern __shared__ __align__(16) float sm[];
    pdl_launch_dependents();
    pdl_wait();
    using L = SBL<D>;
    const int bh = blockIdx.y, h = bh % H, tid = threadIdx.x;
    const int n_tiles = (Tlen + SB_TR - 1) / SB_TR;
    const int tile_begin = blockIdx.x * tiles_per_cta, tile_end = min(tile_begin + tiles_per_cta, n_tiles);
    float* my_part = part + ((size_t)bh * gridDim.x + blockIdx.x) * L::PART_PAD;

    // ---- this head's parameters: weights as [tap][c_in][c_out + 4] ----
    const float* g0 = wpack + (size_t)h * L::G0;
    const float* g1 = wpack + (size_t)H * L::G0 + (size_t)h * L::G1;
    const float* g2 = wpack + (size_t)H * (L::G0 + L::G1) + (size_t)h * L::G2;
    const float* go = wpack + (size_t)H * (L::G0 + L::G1 + L::G2) + (size_t)h * L::C3;
    for (int e = tid; e < L::G0; e += SB_NT) {                 // e = (o * 3 + tau) * C0 + c
        const int c = e % L::C0, ot = e / L::C0, tau = ot % 3, o = ot / 3;
        sm[L::OFF_W0 + (tau * L::C0 + c) * (L::C1 + 4) + o] = g0[e];
    }
    for (int e = tid; e < L::G1; e += SB_NT) {
        const int c = e % L::C1, ot = e / L::C1, tau = ot % 3, o = ot / 3;
        sm[L::OFF_W1 + (tau * L::C1 + c) * (L::C2 + 4) + o] = g1[e];
    }
    for (int e = tid; e < L::G2; e += SB_NT) {
        const int c = e % L::C2, ot = e / L::C2, tau = ot % 3, o = ot / 3;
        sm[L::OFF_W2 + (tau * L::C2 + c) * (L::C3 + 4) + o] = g2[e];
    }
    for (int e = tid; e < L::NP; e += SB_NT) {
        float b = 0.f;
        if (e < L::P1) b = bpack ? bpack[(size_t)h * L::C1 + e] : 0.f;
        else if (e < L::P2) b = bpack ? bpack[(size_t)H * L::C1 + (size_t)h * L::C2 + (e - L::P1)] : 0.f;
        else if (e < L::P3) b = bpack ? bpack[(size_t)H * (L::C1 + L::C2) + (size_t)h * L::C3 + (e - L::P2)] : 0.f;
        else if (e < L::P4) b = go[e - L::P3];
        else b = bpack ? bpack[(size_t)H * (L::C1 + L::C2 + L::C3) + h] : 0.f;
        sm[L::OFF_P + e] = b;
    }
    const float* sb0 = sm + L::OFF_P, *sb1 = sm + L::OFF_P + L::P1, *sb2 = sm + L::OFF_P + L::P2, *swo = sm + L::OFF_P + L::P3;

    // gradient accumulators of this CTA (registers, across its tiles)
    float a0[3][4][L::CB0], a1[3][4][L::CB1], a2[3][4][L::CB2];
#pragma unroll
    for (int t = 0; t < 3; ++t)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
            for (int c = 0; c < L::CB0; ++c) a0[t][j][c] = 0.f;
#pragma unroll
            for (int c = 0; c < L::CB1; ++c) a1[t][j][c] = 0.f;
            a2[t][j][0] = 0.f;
        }
    float small = 0.f;                                         // thread < P1: db0; < P2: db1; < P3: db2; < P4: dwout; P4: dbout

    const T* kk = k + (size_t)bh * Tlen * D;
    const T* vv = v + (size_t)bh * Tlen * D;
    const float* dzz = dz + (size_t)bh * Tlen;
    for (int tile = tile_begin; tile < tile_end; ++tile) {
        const int a = tile * SB_TR;                            // the tile owns times a .. a + TR - 1
        __syncthreads();                                       // the previous tile's readers are done (and the parameters are in)
        // ---- input rows a-12 .. a+TR+11 (zero outside [0, T)) and delta3[t] = dz[t - 6] for the rows a .. a+TR+11 ----
        for (int e = tid; e < SB_RX * (L::C0 / 4); e += SB_NT) {
            const int r = e / (L::C0 / 4), c4 = (e % (L::C0 / 4)) * 4;
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
            *reinterpret_cast<float4*>(&sm[L::OFF_X + r * L::SX + c4]) = x;
        }
        if (tid < SB_R2) {
            const int t = a + tid;
            sm[L::OFF_DZ + tid] = (t >= 6 && t < Tlen) ? dzz[t - 6] : 0.f;   // the caller's dz is zero where the logit is undefined
        }
        __syncthreads();
        // ---- forward, keeping activations and Swish' ----
        sb_forward<L::C0, L::C1, SB_R0, L::SX, L::S0>(sm + L::OFF_X, sm + L::OFF_H0, sm + L::OFF_D0, sm + L::OFF_W0, sb0, a - 8);
        __syncthreads();
        sb_forward<L::C1, L::C2, SB_R1, L::S0, L::S1>(sm + L::OFF_H0, sm + L::OFF_H1, sm + L::OFF_D1, sm + L::OFF_W1, sb1, a - 4);
        __syncthreads();
        sb_forward<L::C2, L::C3, SB_R2, L::S1, L::S2>(sm + L::OFF_H1, sm + L::OFF_H2, sm + L::OFF_D2, sm + L::OFF_W2, sb2, a);
        __syncthreads();
        // ---- output map: dwout, dbout over the tile's own times; delta2 = delta3 wout Swish'(y2) in place ----
        if (tid >= L::P3 && tid <= L::P4) {
            for (int t = 0; t < SB_TR; ++t) {
                const float d3 = sm[L::OFF_DZ + t];
                small += tid == L::P4 ? d3 : d3 * sm[L::OFF_H2 + t * L::S2 + (tid - L::P3)];
            }
        }
        __syncthreads();
        for (int e = tid; e < SB_R2 * L::C3; e += SB_NT) {
            const int r = e / L::C3, c = e % L::C3;
            sm[L::OFF_D2 + r * L::S2 + c] *= sm[L::OFF_DZ + r] * swo[c];
        }
        __syncthreads();
        // ---- layer 2: weight gradient (delta2 x h1), bias, then delta1 into the Swish' buffer of layer 1 (rows from a) ----
        sb_wgrad<L::C3, L::C2, L::CB2, L::S2, L::S1>(a2, sm + L::OFF_D2, sm + L::OFF_H1);
        if (tid >= L::P2 && tid < L::P3)
            for (int t = 0; t < SB_TR; ++t) small += sm[L::OFF_D2 + t * L::S2 + (tid - L::P2)];
        sb_transposed<L::C3, L::C2, SB_TR + 8, L::S2>(sm + L::OFF_D2, sm + L::OFF_W2,
                                                      [&](int r, int c, float g) { sm[L::OFF_D1 + (r + 4) * L::S1 + c] *= g; });
        __syncthreads();
        // ---- layer 1 ----
        sb_wgrad<L::C2, L::C1, L::CB1, L::S1, L::S0>(a1, sm + L::OFF_D1 + 4 * L::S1, sm + L::OFF_H0 + 4 * L::S0);
        if (tid >= L::P1 && tid < L::P2)
            for (int t = 0; t < SB_TR; ++t) small += sm[L::OFF_D1 + (t + 4) * L::S1 + (tid - L::P1)];
        sb_transposed<L::C2, L::C1, SB_TR + 4, L::S1>(sm + L::OFF_D1 + 4 * L::S1, sm + L::OFF_W1,
                                                      [&](int r, int c, float g) { sm[L::OFF_D0 + (r + 8) * L::S0 + c] *= g; });
        __syncthreads();
        // ---- layer 0 ----
        sb_wgrad<L::C1, L::C0, L::CB0, L::S0, L::SX>(a0, sm + L::OFF_D0 + 8 * L::S0, sm + L::OFF_X + 8 * L::SX);
        if (tid < L::P1)
            for (int t = 0; t < SB_TR; ++t) small += sm[L::OFF_D0 + (t + 8) * L::S0 + tid];
        if (input_grad) {
            // the gradient into the inputs: channels [0, 64) into dk, [64, 128) into dv, added to what the attention left there
            sb_transposed<L::C1, L::C0, SB_TR, L::S0>(sm + L::OFF_D0 + 8 * L::S0, sm + L::OFF_W0, [&](int r, int c, float g) {
                const int t = a + r;
                if (t < Tlen) {
                    T* dst = (c < D ? dk : dv) + ((size_t)bh * Tlen + t) * D + (c < D ? c : c - D);
                    *dst = from_f<T>(to_f(*dst) + g);
                }
            });
        }
    }
    // ---- this CTA's partial sums, in the packed layout of the parameters (thread -> block as in sb_wgrad) ----
    {
        constexpr int NCB = L::C0 / L::CB0;                    // layer 0: blocks of 4 outputs x CB0 inputs
        if (tid < (L::C1 / 4) * NCB) {
            const int cb = tid % NCB, ob = tid / NCB;
#pragma unroll
            for (int tau = 0; tau < 3; ++tau)
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int cc = 0; cc < L::CB0; ++cc) my_part[((4 * ob + j) * 3 + tau) * L::C0 + cb * L::CB0 + cc] = a0[tau][j][cc];
        }
    }
    {
        constexpr int NCB = L::C1 / L::CB1;                    // layer 1
        if (tid < (L::C2 / 4) * NCB) {
            const int cb = tid % NCB, ob = tid / NCB;
#pragma unroll
            for (int tau = 0; tau < 3; ++tau)
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int cc = 0; cc < L::CB1; ++cc) my_part[L::G0 + ((4 * ob + j) * 3 + tau) * L::C1 + cb * L::CB1 + cc] = a1[tau][j][cc];
        }
    }
    {
        constexpr int NCB = L::C2 / L::CB2;                    // layer 2
        if (tid < (L::C3 / 4) * NCB) {
            const int cb = tid % NCB, ob = tid / NCB;
#pragma unroll
            for (int tau = 0; tau < 3; ++tau)
#pragma unroll
                for (int j = 0; j < 4; ++j) my_part[L::G0 + L::G1 + ((4 * ob + j) * 3 + tau) * L::C2 + cb] = a2[tau][j][0];
        }
    }
    {
        // wout [C3] | b0 [C1] | b1 [C2] | b2 [C3] | bout
        float* sp = my_part + L::G0 + L::G1 + L::G2;
        if (tid < L::P1) sp[L::C3 + tid] = small;
        else if (tid < L::P2) sp[L::C3 + L::C1 + (tid - L::P1)] = small;
        else if (tid < L::P3) sp[L::C3 + L::C1 + L::C2 + (tid - L::P2)] = small;
        else if (tid < L::P4) sp[tid - L::P3] = small;
        else if (tid == L::P4) sp[L::C3 + L::C1 + L::C2 + L::C3] = small;
    }
}

// dw = wl0 | wl1 | wl2 | wout (every tensor over all heads), dbias = bl0 | bl1 | bl2 | bout: sums of the partials of a head's
// CTAs (all batch elements, all row chunks) in a fixed order.
template <int D>
__global__ void stack_bwd_reduce_kernel(const float* __restrict__ part, float* __restrict__ dw, float* __restrict__ dbias,
                                        int B, int H, int chunks)
{
    using L = SBL<D>;
    pdl_launch_dependents();
    pdl_wait();
    const int h = blockIdx.y, e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= L::PART) return;
    float t = 0.f;
    for (int b = 0; b < B; ++b)
        for (int ch = 0; ch < chunks; ++ch) t += part[(((size_t)b * H + h) * chunks + ch) * L::PART_PAD + e];
    constexpr int GW = L::G0 + L::G1 + L::G2;
    if (e < L::G0) dw[(size_t)h * L::G0 + e] = t;
    else if (e < L::G0 + L::G1) dw[(size_t)H * L::G0 + (size_t)h * L::G1 + (e - L::G0)] = t;
    else if (e < GW) dw[(size_t)H * (L::G0 + L::G1) + (size_t)h * L::G2 + (e - L::G0 - L::G1)] = t;
    else if (e < GW + L::C3) dw[(size_t)H * GW + (size_t)h * L::C3 + (e - GW)] = t;
    else if (dbias) {
        const int f = e - (GW + L::C3);                        // b0 [C1] | b1 [C2] | b2 [C3] | bout
        if (f < L::P1) dbias[(size_t)h * L::C1 + f] = t;
        else if (f < L::P2) dbias[(size_t)H * L::C1 + (size_t)h * L::C2 + (f - L::P1)] = t;
        else if (f < L::P3) dbias[(size_t)H * (L::C1 + L::C2) + (size_t)h * L::C3 + (f - L::P2)] = t;
        else dbias[(size_t)H * (L::C1 + L::C2 + L::C3) + h] = t;
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
    if (p.d != 64 && p.d != 32) return 0;
    const int pad = p.d == 64 ? SBL<64>::PART_PAD : SBL<32>::PART_PAD;
    return (size_t)p.B * p.H * stack_bwd_chunks(p) * pad * sizeof(float);
}

namespace {
template <typename T, int D>
int run_stack_bwd(const Params& p, const void* k, const void* v, const float* dz, void* dk, void* dv, float* dw, float* dbias,
                  bool input_grad, void* part, cudaStream_t st)
{
    using L = SBL<D>;
    const int chunks = stack_bwd_chunks(p);
    const int n_tiles = (p.T + SB_TR - 1) / SB_TR, per = (n_tiles + chunks - 1) / chunks;
    dim3 grid(chunks, p.B * p.H);
    static PerDeviceOnce attr;
    if (int e2 = attr.run([] { return cudaFuncSetAttribute(stack_bwd_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::BYTES); }))
        return e2;
    if (launch_pdl(stack_bwd_kernel<T, D>, grid, dim3(SB_NT), L::BYTES, st, (const T*)k, (const T*)v, p.w, p.bias, dz, (T*)dk, (T*)dv,
                   (float*)part, p.H, p.T, per, input_grad ? 1 : 0) != cudaSuccess)
        return LTE_ERR_CUDA;
    if (launch_pdl(stack_bwd_reduce_kernel<D>, dim3((L::PART + 255) / 256, p.H), dim3(256), 0, st, (const float*)part, dw, dbias, p.B,
                   p.H, chunks) != cudaSuccess)
        return LTE_ERR_CUDA;
    return cuda_status(cudaGetLastError());
}
}  // namespace

// dz [B,H,T] fp32 (zero where the logit is undefined) -> dw, dbias (packed like the parameters; dbias may be null) and,
// with input_grad, dk += , dv += the gradient into the scorer's inputs.  part: stack_bwd_workspace(p) bytes.
int launch_stack_bwd(const Params& p, const void* k, const void* v, const float* dz, void* dk, void* dv, float* dw,
                     float* dbias, bool input_grad, void* part, cudaStream_t st)
{
    const bool bf = p.dtype == LTE_BF16;
    if (p.d == 64)
        return bf ? run_stack_bwd<__nv_bfloat16, 64>(p, k, v, dz, dk, dv, dw, dbias, input_grad, part, st)
                  : run_stack_bwd<float, 64>(p, k, v, dz, dk, dv, dw, dbias, input_grad, part, st);
    if (p.d == 32)
        return bf ? run_stack_bwd<__nv_bfloat16, 32>(p, k, v, dz, dk, dv, dw, dbias, input_grad, part, st)
                  : run_stack_bwd<float, 32>(p, k, v, dz, dk, dv, dw, dbias, input_grad, part, st);
    return LTE_ERR_UNSUPPORTED;
}

}  // namespace lte
