// moesched_bvn_decompose_static: the Birkhoff-von Neumann entry point for callers that
// cannot obtain device memory themselves. Its working copy of the matrices lives in a
// fixed array that is part of the library image, so the call allocates nothing.
#include <mutex>

#include "common.cuh"

namespace moesched {

// Working copy for the batch: B * N * roundup(N, 8) int32 values must fit.
// Every GPU on which the library is loaded reserves this much memory until the process ends.
constexpr size_t STATIC_SCRATCH_INTS = MOESCHED_STATIC_SCRATCH_BYTES / sizeof(int32_t);
static __device__ __align__(256) int32_t g_static_scratch[STATIC_SCRATCH_INTS];

constexpr int MAX_DEVICES = 64;
static std::mutex g_setup_mutex;
static int32_t* g_scratch_addr[MAX_DEVICES];   // device address of the array, per device; null = not set up

// In host code the name g_static_scratch is only a handle for the runtime, not an address a
// kernel could use; the device address has to be asked for, once per device, with that
// device current.
static cudaError_t scratch_address(int32_t** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = static_cast<int32_t*>(p);
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

int& last_cuda_error_slot();

}  // namespace moesched

using namespace moesched;

extern "C" int moesched_bvn_decompose_static(int B, int N, const int32_t* d_demand, int k_max, uint8_t* d_perm,
                                             int32_t* d_coef, int32_t* d_count, int32_t* d_aug,
                                             int32_t* d_status, int64_t* d_work, void* stream) {
  if (B < 0 || N < 1 || N > MOESCHED_MAX_N || k_max < 1) return MOESCHED_EINVAL;
  if (B == 0) return MOESCHED_OK;
  if (!d_demand || !d_perm || !d_coef || !d_count || !d_status) return MOESCHED_EINVAL;
  const uintptr_t misaligned = (reinterpret_cast<uintptr_t>(d_demand) | reinterpret_cast<uintptr_t>(d_coef) |
                                reinterpret_cast<uintptr_t>(d_count) | reinterpret_cast<uintptr_t>(d_status) |
                                reinterpret_cast<uintptr_t>(d_aug)) & 3;
  if (misaligned || (reinterpret_cast<uintptr_t>(d_work) & 7)) return MOESCHED_EINVAL;
  const size_t need = (size_t)B * N * bvn_scratch_stride(N);
  if (need > STATIC_SCRATCH_INTS) return MOESCHED_ETOOBIG;
  int32_t* scratch = nullptr;
  cudaError_t e = scratch_address(&scratch);
  if (e == cudaSuccess)
    e = run_bvn(B, N, d_demand, k_max, d_perm, d_coef, d_count, d_aug, scratch, d_status,
                reinterpret_cast<long long*>(d_work), static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) {
    last_cuda_error_slot() = (int)e;
    return MOESCHED_ECUDA;
  }
  return MOESCHED_OK;
}
