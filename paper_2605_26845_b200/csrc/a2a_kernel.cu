// Idealised congestion-free all-to-all (paper Sec. 4.1 "Comparisons"): the busiest port sets the
// exchange time. One warp streams one matrix from global memory: each lane keeps the sums of the
// columns lane, lane+32, ...; a row sum is one warp reduction per row. The kernel reads every
// entry exactly once and is bound by HBM bandwidth.
#include "common.cuh"

namespace moesched {

constexpr int A2A_WARPS = 8;

// K = column chunks of 32 per row (1, 2, 4 or 8); 32 / K rows are in flight per lane
template <int K>
__global__ void __launch_bounds__(32 * A2A_WARPS) ideal_a2a_kernel(int B, int N, const int32_t* __restrict__ demand,
                                                                   moesched_model_t model,
                                                                   long long* __restrict__ comm_ns,
                                                                   long long* __restrict__ makespan_ns,
                                                                   int32_t* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * A2A_WARPS + (threadIdx.x >> 5);
  if (b >= B) return;
  const int32_t* D = demand + (size_t)b * N * N;
  long long col[K];
#pragma unroll
  for (int k = 0; k < K; ++k) col[k] = 0;
  long long rowmax = 0;
  int neg = 0;
  constexpr int UNROLL = 32 / K;   // rows in flight per lane: their loads do not depend on one another
  for (int r0 = 0; r0 < N; r0 += UNROLL) {
    int v[UNROLL][K];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
#pragma unroll
      for (int k = 0; k < K; ++k) {
        const int c = lane + 32 * k;
        v[u][k] = (r0 + u < N && c < N) ? D[(size_t)(r0 + u) * N + c] : 0;
      }
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      // exact row sum from two 32-bit warp additions: low and high halves of the entries
      unsigned lo = 0u, hi = 0u;
#pragma unroll
      for (int k = 0; k < K; ++k) {
        neg |= v[u][k] < 0;
        col[k] += v[u][k];
        lo += (unsigned)v[u][k] & 0xffffu;
        hi += (unsigned)v[u][k] >> 16;
      }
      lo = __reduce_add_sync(FULL, lo);
      hi = __reduce_add_sync(FULL, hi);
      rowmax = max(rowmax, ((long long)hi << 16) + lo);
    }
  }
  long long colmax = 0;
#pragma unroll
  for (int k = 0; k < K; ++k) colmax = max(colmax, col[k]);
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
  if (N <= 32) ideal_a2a_kernel<1><<<blocks, 32 * A2A_WARPS, 0, stream>>>(B, N, demand, model, comm_ns, makespan_ns, status);
  else if (N <= 64) ideal_a2a_kernel<2><<<blocks, 32 * A2A_WARPS, 0, stream>>>(B, N, demand, model, comm_ns, makespan_ns, status);
  else if (N <= 128) ideal_a2a_kernel<4><<<blocks, 32 * A2A_WARPS, 0, stream>>>(B, N, demand, model, comm_ns, makespan_ns, status);
  else ideal_a2a_kernel<8><<<blocks, 32 * A2A_WARPS, 0, stream>>>(B, N, demand, model, comm_ns, makespan_ns, status);
  return cudaGetLastError();
}

}  // namespace moesched
