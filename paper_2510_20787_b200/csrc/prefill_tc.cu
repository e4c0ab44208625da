// placeholder until the tensor-core kernel lands: bf16 prefill runs on the fp32-ALU kernel
#include "common.cuh"
namespace lte {
int launch_prefill_tc(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx,
                      const int32_t* cnt, void* o, float* lse, cudaStream_t st)
{
    return launch_prefill_simt(p, q, k, v, idx, cnt, o, lse, st);
}
}  // namespace lte
