// Idealised congestion-free all-to-all (paper Sec. 4.1 "Comparisons"): the busiest port sets the
// exchange time. One warp streams one matrix from global memory: each lane keeps the sums of the
// columns lane, lane+32, ...; a row sum is one warp reduction per row. The kernel reads every
// entry exactly once and is bound by HBM bandwidth.
#include "common.cuh"

namespace moesched {

constexpr int A2A_WARPS = 8;

__global__ void __launch_bounds__(32 * A2A_WARPS) ideal_a2a_kernel(int B, int N, const int32_t* __restrict__ demand,
                                                                   moesched_model_t model,
                                                                   long long* __restrict__ comm_ns,
                                                                   long long* __restrict__ makespan_ns,
                                                                   int32_t* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * A2A_WARPS + (threadIdx.x >> 5);
  if (b >= B) return;
  const int32_t* D = demand + (size_t)b * N * N;
  long long col[MOESCHED_MAX_N / 32];
#pragma unroll
  for (int k = 0; k < MOESCHED_MAX_N / 32; ++k) col[k] = 0;
  long long rowmax = 0;
  int neg = 0;
  for (int r = 0; r < N; ++r) {
    long long part = 0;
#pragma unroll
    for (int k = 0; k < MOESCHED_MAX_N / 32; ++k) {
      const int c = lane + 32 * k;
      if (c < N) {
        const int v = D[(size_t)r * N + c];
        neg |= v < 0;
        col[k] += v;
        part += v;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(FULL, part, o);
    rowmax = max(rowmax, part);
  }
  long long colmax = 0;
#pragma unroll
  for (int k = 0; k < MOESCHED_MAX_N / 32; ++k) colmax = max(colmax, col[k]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) colmax = max(colmax, __shfl_xor_sync(FULL, colmax, o));
  neg = __any_sync(FULL, neg);
  const long long port = max(rowmax, colmax);
  if (lane == 0) {
    if (neg || port > 2147483647LL) {
      comm_ns[b] = 0;
      makespan_ns[b] = 0;
      status[b] = MOESCHED_ST_BAD_INPUT;
    } else {
      const long long t = (port * model.bytes_per_token * 8 + model.link_gbps - 1) / model.link_gbps;
      comm_ns[b] = t;
      makespan_ns[b] = 2 * t + batch_time_ns(model, colmax);
      status[b] = MOESCHED_ST_OK;
    }
  }
}

cudaError_t run_ideal_a2a(int B, int N, const int32_t* demand, const moesched_model_t& model, long long* comm_ns,
                          long long* makespan_ns, int32_t* status, cudaStream_t stream) {
  const int blocks = (B + A2A_WARPS - 1) / A2A_WARPS;
  ideal_a2a_kernel<<<blocks, 32 * A2A_WARPS, 0, stream>>>(B, N, demand, model, comm_ns, makespan_ns, status);
  return cudaGetLastError();
}

}  // namespace moesched
