// Shared device/host helpers of liblte (CUDA side only; the CPU oracle shares nothing with this).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <mutex>

#include "lte.h"

namespace lte {

constexpr int kMaxTaps = 13;          // scorer taps the kernels are instantiated for (odd, <= 13)

struct Params {                       // validated, host-resolved view of lte_shape / lte_conv
    int B, H, T, d, W, R, sink, K, half;
    int G;                            // query heads per key/value head (q, o, lse have H * G heads)
    int qoff;                         // prefill attention: q, o, lse hold the queries at positions qoff .. T-1 only (chunked prefill; else 0)
    int stack;                        // 1: the three-layer scorer stack (w, bias packed as lte.h describes; K = 13, half = 6)
    float zthr;                       // logit(tau): keep iff z > zthr
    float scale;                      // softmax scale
    int dtype;
    const float* w;
    const float* bias;
};

template <typename T> __device__ __forceinline__ float to_f(T x);
template <> __device__ __forceinline__ float to_f<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}

// Monotone image of an fp32 logit: larger z <=> larger key.  0 is reserved for "not a candidate".
__device__ __forceinline__ uint32_t order_key(float z) {
    uint32_t u = __float_as_uint(z);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// ---- decode cache layout (per (b,h) block; see lte_cache_bytes) -----------------------------
struct CacheLayout {
    size_t esz;            // element size of k/v
    size_t off_k, off_v;   // [rows_alloc, d] each: rows [0,W) ring (slot = pos mod W), rows [W,W+R) pool
    size_t off_z;          // [(W+R)] fp32 logits, same row order
    size_t off_pidx;       // [R] int32 positions of pool entries
    size_t off_meta;       // int32[4]: n (tokens seen), cnt (pool entries), reserved x2
    size_t stride;         // bytes per (b,h), multiple of 256
    size_t header;         // bytes before the first (b,h) block (status word lives at byte 0)
    int rows_alloc;        // key/value rows per block (W+R, or 256 with zero rows at the end in the swizzled layout)
    int swz;               // 1: bf16, d = 64, W+R <= 256: rows are stored with the 128-byte swizzle (16-byte chunk c of
                           //    row r sits at chunk position c ^ (r & 7)) so that the block, once copied to shared memory,
                           //    is a valid tcgen05 operand as it stands
};
__host__ __device__ inline CacheLayout cache_layout(int d, int W, int R, int dtype) {
    CacheLayout L;
    L.esz = dtype == LTE_BF16 ? 2 : 4;
    L.swz = (dtype == LTE_BF16 && d == 64 && W + R <= 256) ? 1 : 0;
    L.rows_alloc = L.swz ? 256 : W + R;
    size_t rows = (size_t)W + R;
    L.off_k = 0;
    L.off_v = L.off_k + (size_t)L.rows_alloc * d * L.esz;
    L.off_z = L.off_v + (size_t)L.rows_alloc * d * L.esz;
    L.off_pidx = L.off_z + rows * 4;
    L.off_meta = L.off_pidx + (size_t)R * 4;
    size_t end = L.off_meta + 16;
    L.stride = (end + 255) / 256 * 256;
    L.header = 256;
    return L;
}
// chunk position of logical 16-byte chunk `c` of row `row` (bf16, d = 64: 8 chunks per row)
__host__ __device__ inline int cache_chunk_pos(const CacheLayout& L, int row, int c) { return L.swz ? (c ^ (row & 7)) : c; }

// kernel launchers (one translation unit each)
int launch_scores(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st);
int launch_scores_stack(const Params& p, const void* k, const void* v, float* z, float* r, cudaStream_t st);
size_t scores_stack_weight_floats(int d, int H);
size_t scores_stack_tc_workspace(const Params& p);
size_t stack_bwd_workspace(const Params& p);
size_t stack_bwd_tc_workspace(const Params& p);
int launch_stack_bwd_tc(const Params& p, const void* k, const void* v, const float* dz, void* dk, void* dv, float* dw,
                        float* dbias, bool input_grad, void* ws, cudaStream_t st);
int launch_stack_bwd(const Params& p, const void* k, const void* v, const float* dz, void* dk, void* dv, float* dw,
                     float* dbias, bool input_grad, void* part, cudaStream_t st);
int launch_scores_stack_tc(const Params& p, const void* k, const void* v, float* z, float* r, void* ws, size_t ws_bytes,
                           cudaStream_t st);
int launch_select(const Params& p, const float* z, int32_t* idx, int32_t* cnt, int32_t* ncand, cudaStream_t st);
int launch_select_uniform(const Params& p, int32_t* idx, int32_t* cnt, int32_t* ncand, cudaStream_t st);
int launch_colsum(const Params& p, const void* q, const void* k, const float* lse, const int32_t* idx, const int32_t* cnt,
                  float* a, cudaStream_t st);
int launch_prefill_simt(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx,
                        const int32_t* cnt, void* o, float* lse, cudaStream_t st, const int32_t* leave = nullptr);
int launch_chunk_stream(const Params& p, const float* zrank, const int32_t* oldpos, int32_t* ulist, int32_t* leave, int32_t* ucnt,
                        int32_t* idx, int32_t* cnt, int ucap, int n0, int R0, int Wn, cudaStream_t st);
int launch_prefill_tc_long(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx,
                           const int32_t* cnt, void* o, float* lse, void* ws, size_t ws_bytes, cudaStream_t st,
                           const int32_t* leave = nullptr);
size_t prefill_compact_bytes(const Params& p);
int launch_prefill_compact(const Params& p, const void* k, const void* v, const int32_t* idx, const int32_t* cnt, void* kc, void* vc,
                           cudaStream_t st);
int prefill_long_status_fetch_and_clear();
int launch_cache_init(const Params& p, const void* k, const void* v, const float* z, const int32_t* idx,
                      const int32_t* cnt, void* cache, cudaStream_t st);
int launch_ring_linearize(const Params& p, const void* cache, void* klin, void* vlin, const float* rope_cos, const float* rope_sin,
                          int rope_len, cudaStream_t st);
int launch_ring_scatter_z(const Params& p, void* cache, const float* zlin, cudaStream_t st);
int launch_chunk_gather(const Params& p, const void* cache, const void* k, const void* v, void* klin, void* vlin, float* zsrc,
                        int32_t* oldpos, int32_t* gate, int n0, int R0, int Wn, cudaStream_t st);
int launch_chunk_merge_z(const Params& p, float* z, float* zrank, const float* zsrc, const int32_t* oldpos, int n0, int R0, int Wn,
                         cudaStream_t st);
int launch_chunk_commit(const Params& p, void* cache, const void* klin, const void* vlin, const float* z, const int32_t* idx,
                        const int32_t* cnt, const int32_t* oldpos, const int32_t* gate, int n0, int n1, int R0, int Wn,
                        cudaStream_t st);
int chunk_status_fetch_and_clear();
int launch_sparsity_stats(const Params& p, const float* z, const float* lambda, float* count, float* penalty, float* part, float tau,
                          cudaStream_t st);
int launch_decode_tc(const Params& p, void* cache, const void* q1, const void* k1, const void* v1, void* o1,
                     float* lse1, cudaStream_t st);
int launch_decode(const Params& p, void* cache, const void* q1, const void* k1, const void* v1, void* o1,
                  float* lse1, cudaStream_t st);
size_t bwd_workspace_bytes(const Params& p, uint32_t flags);
int launch_bwd(const Params& p, const void* q, const void* k, const void* v, const void* o, const float* lse,
               const void* dO, const float* z, const int32_t* idx, const int32_t* cnt, const float* lambda,
               void* dq, void* dk, void* dv, float* dw, float* dbias, uint32_t flags, void* ws,
               cudaStream_t st);

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? LTE_OK : LTE_ERR_CUDA; }

// Device-side status of one kernel family (a __device__ variable per family, so one per device).
//   code        sticky report for the host: 0, or the code of the first anomaly since lte_device_status() last read it
//               (a bounded wait that gave up, a cache in another state than the call said, ...).  Never read by kernels.
//   abort_grid  grid id of the launch whose bounded wait gave up last (~0 = none): only the waits of that same launch
//               look at it, to end the lost launch quickly.  A later launch has another grid id and waits normally.
struct StatusWord { int code; int pad; unsigned long long abort_grid; };
#define LTE_STATUS_INIT {0, 0, ~0ull}
template <typename Sym> inline int status_fetch_and_clear(const Sym& sym)
{
    StatusWord h;
    if (cudaMemcpyFromSymbol(&h, sym, sizeof(h)) != cudaSuccess) return -1;
    if (h.code != 0 || h.abort_grid != ~0ull) {
        const StatusWord z = LTE_STATUS_INIT;
        if (cudaMemcpyToSymbol(sym, &z, sizeof(z)) != cudaSuccess) return -1;
    }
    return h.code;
}

// Host-side facts that belong to a device, not to the process: looked up (or applied) once per device ordinal, under a
// mutex, by whichever thread gets there first with that device current.  `init` returns an lte_status; a failed init
// is retried by the next call.
constexpr int kMaxDevices = 64;
template <typename T> class PerDevice {
public:
    template <typename F> int get(T* out, F&& init)
    {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess) return LTE_ERR_CUDA;
        return get_for(dev, out, init);
    }
    template <typename F> int get_for(int dev, T* out, F&& init)
    {
        if (dev < 0 || dev >= kMaxDevices) return LTE_ERR_UNSUPPORTED;
        std::lock_guard<std::mutex> lock(mu_);
        if (!have_[dev]) {
            const int e = init(&val_[dev]);
            if (e != LTE_OK) return e;
            have_[dev] = true;
        }
        if (out) *out = val_[dev];
        return LTE_OK;
    }
private:
    std::mutex mu_;
    bool have_[kMaxDevices] = {};
    T val_[kMaxDevices] = {};
};
// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) and the like: once per device.  `f` returns a cudaError_t.
class PerDeviceOnce {
public:
    template <typename F> int run(F&& f) { return t_.get(nullptr, [&](char*) { return cuda_status(f()); }); }
private:
    PerDevice<char> t_;
};
int device_sm_count(int* n_sm);       // SM count of the current device

// Programmatic dependent launch: a kernel launched through launch_pdl may become resident while its predecessor in the
// stream is still running, and does its set-up (barriers, tensor memory, index arithmetic) there.  It must execute
// pdl_wait() before it reads anything a predecessor may have written and before its first global write; the wait
// returns once every earlier grid of the stream has completed and its writes are visible.  pdl_launch_dependents()
// lets the successor (if it was launched the same way) start becoming resident.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

}  // namespace lte
