// Integer issue-rate probe: the measured ceiling for the plain add / min / logic work the
// decomposition kernels are made of. Eight independent chains per thread keep every
// scheduler busy; three dependent operations per chain per iteration.
#include "common.cuh"

namespace moesched {

constexpr int PROBE_CHAINS = 8;
constexpr int PROBE_OPS_PER_CHAIN = 3;

__global__ void __launch_bounds__(256) int_probe_kernel(int iters, unsigned seed, unsigned* __restrict__ out) {
  unsigned a[PROBE_CHAINS];
  const unsigned tid = blockIdx.x * blockDim.x + threadIdx.x;
#pragma unroll
  for (int c = 0; c < PROBE_CHAINS; ++c) a[c] = tid * 2654435761u + c * 40503u + seed;
  const unsigned k1 = seed | 1u, k2 = ~seed;
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int c = 0; c < PROBE_CHAINS; ++c) {
      unsigned v = a[c] + k1;          // add
      v = min(v, k2 - c);              // min
      a[c] = v ^ (unsigned)it;         // logic
    }
  }
  unsigned r = 0;
#pragma unroll
  for (int c = 0; c < PROBE_CHAINS; ++c) r ^= a[c];
  out[tid] = r;
}

int& last_cuda_error_slot();

}  // namespace moesched

using namespace moesched;

extern "C" long long moesched_probe_int_ops(int blocks, int iters, uint32_t* d_out, void* stream) {
  if (blocks < 1 || iters < 1 || !d_out || (reinterpret_cast<uintptr_t>(d_out) & 3)) return MOESCHED_EINVAL;
  int_probe_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(iters, 12345u, d_out);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    last_cuda_error_slot() = (int)e;
    return MOESCHED_ECUDA;
  }
  return (long long)blocks * 256 * iters * PROBE_CHAINS * PROBE_OPS_PER_CHAIN;
}
