// The paper's scorer stack on the GPU (Section 3.1.1, hyper-parameters of Appendix A): three dilated grouped conv
// layers (kernel 3, dilation 2) over x = [k ; v], channels 2d -> d -> d/2 -> d/4, each followed by Swish, then a
// per-head linear map to one logit; receptive field 13, the logit of token j is the stack's output at time j + 6.
// Causal form, as the oracle states it: every layer's input (hidden activations included) is zero at negative
// times; there is no right padding, so z_j = -inf for j > T-1-6.
//
// fp32 on the ordinary ALUs, on purpose: the keep decision z > logit(tau) has to agree with an fp64 evaluation to
// within 4e-5 on z, which bf16 tensor-core products of fp32 activations do not give without splitting every
// operand.  A CTA keeps one head's weights (all three layers, transposed to [tap][c_in][c_out]) in shared memory and
// walks row tiles of 64 logits: the input rows with their halo (12 earlier rows), then the three layers as small
// register-tiled products out of shared memory (a thread owns 4 output channels of a few rows; activations are read
// as broadcast 16-byte loads, weights as contiguous ones), then the 64 dot products with the output vector.
#include "common.cuh"

namespace lte {
namespace {

constexpr int SK_KS = 3, SK_DIL = 2, SK_HALF = 6;   // half = L (ks-1) dil / 2
constexpr int SK_TR = 64;                           // logits per tile
constexpr int SK_NT = 256;

template <int D> struct StackPlan {
    static constexpr int C0 = 2 * D, C1 = D, C2 = D / 2, C3 = D / 4;
    static constexpr int R3 = SK_TR, R2 = SK_TR + 4, R1 = SK_TR + 8, R0 = SK_TR + 12;   // rows a layer must provide
    static constexpr int S0 = C0 + 4, S1 = C1 + 4, S2 = C2 + 4;   // padded row strides (floats): conflict-free 16-byte reads
    static constexpr int W1 = SK_KS * C0 * C1, W2 = SK_KS * C1 * C2, W3 = SK_KS * C2 * C3;
    static constexpr int OFF_W1 = 0, OFF_W2 = OFF_W1 + W1, OFF_W3 = OFF_W2 + W2, OFF_WO = OFF_W3 + W3;
    static constexpr int OFF_B = OFF_WO + C3;                      // b1 | b2 | b3 | bout
    static constexpr int OFF_X = (OFF_B + C1 + C2 + C3 + 1 + 3) & ~3;
    static constexpr int OFF_A1 = OFF_X + R0 * S0, OFF_A2 = OFF_A1 + R1 * S1, OFF_A3 = OFF_A2 + R2 * S2;
    static constexpr int FLOATS = OFF_A3 + R3 * C3;
    static constexpr size_t BYTES = (size_t)FLOATS * sizeof(float);
    // packed parameter layout in global memory (per tensor: all heads): wl0 | wl1 | wl2 | wout and bl0 | bl1 | bl2 | bout
    static constexpr int GW1 = C1 * SK_KS * C0, GW2 = C2 * SK_KS * C1, GW3 = C3 * SK_KS * C2;
};

// One layer: out[r][o] = Swish(bias[o] + sum_{tau, c} w[tau][c][o] in[r + tau * DIL][c]) for rows r < ROWS; out row r is
// at time t_out0 + r and is forced to zero when that time is negative.  in row 0 is at time t_out0 - (KS-1) DIL.
template <int CIN, int COUT, int ROWS, int SIN, int SOUT>
__device__ __forceinline__ void stack_layer(const float* __restrict__ in, float* __restrict__ out,
                                            const float* __restrict__ w, const float* __restrict__ bias, int t_out0)
{
    constexpr int TX = COUT / 4, TY = SK_NT / TX, RPT = (ROWS + TY - 1) / TY;
    const int tx = threadIdx.x % TX, ty = threadIdx.x / TX;
    float acc[RPT][4];
#pragma unroll
    for (int i = 0; i < RPT; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
    int rrow[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) rrow[i] = min(ty + TY * i, ROWS - 1);   // surplus threads recompute the last row
#pragma unroll 1
    for (int tau = 0; tau < SK_KS; ++tau) {
#pragma unroll 2
        for (int c = 0; c < CIN; c += 4) {
            float4 a[RPT];
#pragma unroll
            for (int i = 0; i < RPT; ++i) a[i] = *reinterpret_cast<const float4*>(&in[(rrow[i] + tau * SK_DIL) * SIN + c]);
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const float4 b = *reinterpret_cast<const float4*>(&w[((tau * CIN) + c + cc) * COUT + 4 * tx]);
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
            const bool live = t_out0 + r >= 0;
            float y[4] = {acc[i][0] + bb.x, acc[i][1] + bb.y, acc[i][2] + bb.z, acc[i][3] + bb.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) y[e] = live ? y[e] / (1.f + expf(-y[e])) : 0.f;      // Swish
            *reinterpret_cast<float4*>(&out[r * SOUT + 4 * tx]) = make_float4(y[0], y[1], y[2], y[3]);
        }
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(SK_NT, 1)
scores_stack_kernel(const T* __restrict__ k, const T* __restrict__ v, const float* __restrict__ wpack,
                    const float* __restrict__ bpack, float* __restrict__ z, float* __restrict__ r_out, int H, int Tlen,
                    int tiles_per_cta)
{
    using P = StackPlan<D>;
    extern __shared__ __align__(16) float sm[];
    pdl_launch_dependents();
    pdl_wait();
    const int bh = blockIdx.y, h = bh % H, tid = threadIdx.x;
    const int n_tiles = (Tlen + SK_TR - 1) / SK_TR;
    const int tile_begin = blockIdx.x * tiles_per_cta, tile_end = min(tile_begin + tiles_per_cta, n_tiles);
    if (tile_begin >= tile_end) return;

    // ---- this head's parameters, transposed to [tap][c_in][c_out] (o fastest) ---------------------------------
    const float* g1 = wpack + (size_t)h * P::GW1;
    const float* g2 = wpack + (size_t)H * P::GW1 + (size_t)h * P::GW2;
    const float* g3 = wpack + (size_t)H * (P::GW1 + P::GW2) + (size_t)h * P::GW3;
    const float* go = wpack + (size_t)H * (P::GW1 + P::GW2 + P::GW3) + (size_t)h * P::C3;
    for (int e = tid; e < P::W1; e += SK_NT) {                 // e = (tau * C0 + c) * C1 + o
        const int o = e % P::C1, kc = e / P::C1, c = kc % P::C0, tau = kc / P::C0;
        sm[P::OFF_W1 + e] = g1[((size_t)o * SK_KS + tau) * P::C0 + c];
    }
    for (int e = tid; e < P::W2; e += SK_NT) {
        const int o = e % P::C2, kc = e / P::C2, c = kc % P::C1, tau = kc / P::C1;
        sm[P::OFF_W2 + e] = g2[((size_t)o * SK_KS + tau) * P::C1 + c];
    }
    for (int e = tid; e < P::W3; e += SK_NT) {
        const int o = e % P::C3, kc = e / P::C3, c = kc % P::C2, tau = kc / P::C2;
        sm[P::OFF_W3 + e] = g3[((size_t)o * SK_KS + tau) * P::C2 + c];
    }
    for (int e = tid; e < P::C3; e += SK_NT) sm[P::OFF_WO + e] = go[e];
    for (int e = tid; e < P::C1 + P::C2 + P::C3 + 1; e += SK_NT) {
        float b = 0.f;
        if (bpack) {
            if (e < P::C1) b = bpack[(size_t)h * P::C1 + e];
            else if (e < P::C1 + P::C2) b = bpack[(size_t)H * P::C1 + (size_t)h * P::C2 + (e - P::C1)];
            else if (e < P::C1 + P::C2 + P::C3) b = bpack[(size_t)H * (P::C1 + P::C2) + (size_t)h * P::C3 + (e - P::C1 - P::C2)];
            else b = bpack[(size_t)H * (P::C1 + P::C2 + P::C3) + h];
        }
        sm[P::OFF_B + e] = b;
    }

    const T* kk = k + (size_t)bh * Tlen * D;
    const T* vv = v + (size_t)bh * Tlen * D;
    for (int tile = tile_begin; tile < tile_end; ++tile) {
        const int j0 = tile * SK_TR;
        const int tb = j0 + SK_HALF;                           // time of the first layer-3 output of the tile
        __syncthreads();                                       // the previous tile's readers are done (and the parameters are in)
        // input rows tb-12 .. tb+63, zero outside [0, T)
        for (int e = tid; e < P::R0 * (P::C0 / 4); e += SK_NT) {
            const int r = e / (P::C0 / 4), c4 = (e % (P::C0 / 4)) * 4;
            const int t = tb - 12 + r;
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
            *reinterpret_cast<float4*>(&sm[P::OFF_X + r * P::S0 + c4]) = x;
        }
        __syncthreads();
        stack_layer<P::C0, P::C1, P::R1, P::S0, P::S1>(sm + P::OFF_X, sm + P::OFF_A1, sm + P::OFF_W1, sm + P::OFF_B, tb - 8);
        __syncthreads();
        stack_layer<P::C1, P::C2, P::R2, P::S1, P::S2>(sm + P::OFF_A1, sm + P::OFF_A2, sm + P::OFF_W2, sm + P::OFF_B + P::C1, tb - 4);
        __syncthreads();
        stack_layer<P::C2, P::C3, P::R3, P::S2, P::C3>(sm + P::OFF_A2, sm + P::OFF_A3, sm + P::OFF_W3, sm + P::OFF_B + P::C1 + P::C2, tb);
        __syncthreads();
        if (tid < SK_TR) {
            const int j = j0 + tid;
            if (j < Tlen) {
                float zz = -INFINITY;
                if (j + SK_HALF <= Tlen - 1) {
                    zz = sm[P::OFF_B + P::C1 + P::C2 + P::C3];
#pragma unroll
                    for (int c = 0; c < P::C3; ++c) zz = fmaf(sm[P::OFF_WO + c], sm[P::OFF_A3 + tid * P::C3 + c], zz);
                }
                z[(size_t)bh * Tlen + j] = zz;
                if (r_out) r_out[(size_t)bh * Tlen + j] = 1.f / (1.f + expf(-zz));
            }
        }
    }
}

template <typename T, int D>
int run_stack(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    using P = StackPlan<D>;
    static PerDeviceOnce attr;
    if (int e = attr.run([] { return cudaFuncSetAttribute(scores_stack_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)P::BYTES); }))
        return e;
    int sms = 148;
    device_sm_count(&sms);
    const int BH = p.B * p.H, n_tiles = (p.T + SK_TR - 1) / SK_TR;
    // a CTA keeps one head's parameters in shared memory (one CTA per SM): split every (b,h) into about SMs / (B H) chunks
    int chunks = sms / BH;
    if (chunks < 1) chunks = 1;
    if (chunks > n_tiles) chunks = n_tiles;
    const int per = (n_tiles + chunks - 1) / chunks;
    chunks = (n_tiles + per - 1) / per;
    dim3 grid(chunks, BH);
    return cuda_status(launch_pdl(scores_stack_kernel<T, D>, grid, dim3(SK_NT), P::BYTES, st, (const T*)k, (const T*)v, p.w, p.bias,
                                  z, r, p.H, p.T, per));
}

}  // namespace

// Packed parameter sizes of the stack for head dimension d (floats): weights and biases.
size_t scores_stack_weight_floats(int d, int H)
{
    return (size_t)H * ((size_t)d * 3 * 2 * d + (size_t)(d / 2) * 3 * d + (size_t)(d / 4) * 3 * (d / 2) + d / 4);
}

int launch_scores_stack(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st)
{
    if (p.dtype == LTE_BF16) {
        if (p.d == 64) return run_stack<__nv_bfloat16, 64>(p, k, v, z, r, st);
        if (p.d == 32) return run_stack<__nv_bfloat16, 32>(p, k, v, z, r, st);
    } else {
        if (p.d == 64) return run_stack<float, 64>(p, k, v, z, r, st);
        if (p.d == 32) return run_stack<float, 32>(p, k, v, z, r, st);
    }
    return LTE_ERR_UNSUPPORTED;                                // d = 128: the first layer's weights alone exceed shared memory
}

}  // namespace lte
