// firp_topb_static: the two-pass top-B of logits rows with its candidate scratch in a static device
// array, for callers that must not allocate device memory.  (The paper has no counterpart.)
#include <cstdio>
#include <mutex>

#include "../../include/firp.h"
#include "firp_kernels.cuh"

namespace {

// Candidate scratch of pass 1: one slot of kMaxTopB (id, value) pairs per (row, 2048-logit segment).
// 256 KiB, held by every GPU that loads the library until the process exits.
constexpr int kStaticSlots = FIRP_TOPB_STATIC_MAX_SLOTS;
static __device__ __align__(256) unsigned char g_topb_scratch[(size_t)kStaticSlots * firp::kMaxTopB * 8];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void *g_scratch_addr[kMaxDevices];   // device address of g_topb_scratch on each device, once looked up

// In host code `g_topb_scratch` names a host-side shadow of the array, not device memory: the device
// address has to be asked for, on the device it is wanted for.
cudaError_t scratch_address(void **out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_topb_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int firp_topb_static(const float *d_logits, int32_t rows, int32_t vocab, int32_t b, int32_t *d_ids,
                                float *d_vals, void *stream) {
  if (!d_logits || !d_ids || !d_vals || rows < 1 || vocab < 1 || b < 1 || b > firp::kMaxTopB) {
    fprintf(stderr, "firp_topb_static: NULL pointer, or rows / vocab / b out of range (b must be 1..%d)\n", firp::kMaxTopB);
    return FIRP_ERR_BAD_ARG;
  }
  // segment count in 64 bits: (vocab + 2047) would wrap for a vocab next to INT32_MAX
  const long long slots = (long long)rows * (((long long)vocab + firp::kTopSeg - 1) / firp::kTopSeg);
  if (slots > kStaticSlots) {
    fprintf(stderr, "firp_topb_static: rows * ceil(vocab / 2048) = %lld exceeds the built-in scratch of %d slots\n", slots,
            kStaticSlots);
    return FIRP_ERR_CAPACITY;
  }
  void *scratch = nullptr;
  cudaError_t e = scratch_address(&scratch);
  if (e != cudaSuccess) {
    fprintf(stderr, "firp_topb_static: cudaGetSymbolAddress: %s\n", cudaGetErrorString(e));
    return FIRP_ERR_CUDA;
  }
  // ids in the first half of the array, values in the second; every slot the second pass reads is written
  // by the first pass of the same call, so nothing has to be cleared
  int32_t *cand_ids = reinterpret_cast<int32_t *>(scratch);
  float *cand_vals = reinterpret_cast<float *>(static_cast<unsigned char *>(scratch) + (size_t)kStaticSlots * firp::kMaxTopB * 4);
  firp::launch_topb(d_logits, rows, vocab, b, cand_ids, cand_vals, d_ids, d_vals, false, (cudaStream_t)stream);
  e = cudaGetLastError();
  if (e != cudaSuccess) {
    fprintf(stderr, "firp_topb_static: launch failed: %s\n", cudaGetErrorString(e));
    return FIRP_ERR_CUDA;
  }
  return FIRP_OK;
}
