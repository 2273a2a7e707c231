// Finishers of the stream-K GEMMs as kernels of their own (the bodies live in finish_device.cuh).  The kernels
// use no shared memory and few registers: they stay resident beside the next GEMM's CTAs, whose weight stream
// therefore runs while they work.
#include "finish_device.cuh"
#include "firp_kernels.cuh"
#include "launch_util.cuh"

namespace firp {

namespace {

constexpr int kThreads = 256;

#define FIRP_FINISH_KERNEL(name, minblocks)                                                                     \
  __global__ void __launch_bounds__(kThreads, minblocks) name##_kernel(Partials p, GemmArgs a, int n_st, int pdl) { \
    if (pdl) { griddep_launch(); griddep_wait(); }                                                                \
    name##_item(p, a, n_st, blockIdx.x * blockDim.x + threadIdx.x);                                               \
  }
FIRP_FINISH_KERNEL(qkv_finish, 5)
FIRP_FINISH_KERNEL(swiglu_finish, 5)
FIRP_FINISH_KERNEL(logits_finish, 1)
FIRP_FINISH_KERNEL(pseudo_finish, 1)
#undef FIRP_FINISH_KERNEL

}  // namespace

cudaError_t launch_gemm_finish(GemmEpilogue epi, const Partials &p, const GemmArgs &a, bool pdl, cudaStream_t st) {
  const int n_st = p.sk.U / p.sk.KB;
  const long long threads = (long long)n_st * a.R * 32;
  const dim3 grid((unsigned)((threads + kThreads - 1) / kThreads)), block(kThreads);
  switch (epi) {
    case EPI_QKV_ROPE: return launch_k(qkv_finish_kernel, grid, block, 0, st, pdl, p, a, n_st, pdl ? 1 : 0);
    case EPI_SWIGLU: return launch_k(swiglu_finish_kernel, grid, block, 0, st, pdl, p, a, n_st, pdl ? 1 : 0);
    case EPI_LOGITS: return launch_k(logits_finish_kernel, grid, block, 0, st, pdl, p, a, n_st, pdl ? 1 : 0);
    case EPI_PSEUDO: return launch_k(pseudo_finish_kernel, grid, block, 0, st, pdl, p, a, n_st, pdl ? 1 : 0);
    default: return cudaErrorInvalidValue;   // the residual GEMMs are finished by the RMSNorm kernel
  }
}

}  // namespace firp
