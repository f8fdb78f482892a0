// Order of the matchings and budget choice (paper Sec. 3.3: dispatch, expert compute and combine are
// the three machines of a flow shop, and the order of the matchings changes the makespan; the paper
// leaves the rule open). One warp per schedule.
//
// The job times a_k = reconfiguration + transfer time and b_k = expert batch time come from the
// scoring kernel's replay in emission order. Five candidate orders are built by rank sorting (every
// job counts the jobs that precede it under the candidate's key, ties by the lower original index)
// and each is run through the three-stage recurrence by one lane; the shortest wins, the lower rule
// number on ties:
//   0 emission order; 1 Johnson's rule on stages one and two (a <= b first by increasing a, then the
//   rest by decreasing b); 2 the same on stages two and three (b <= a first by increasing b, then the
//   rest by decreasing a); 3 increasing a placed alternately at the front and at the back; 4 decreasing b.
#include "common.cuh"

namespace moesched {

namespace {

constexpr int ORDER_RULES = 5;
constexpr unsigned long long KEY_TOP = 1ull << 60;   // above every time the input ranges allow

struct JobKeys {
  unsigned long long k1, k2, k3, k4;
};

// Sort keys of one job under the four non-trivial rules (ascending order of the key = schedule order).
__device__ __forceinline__ JobKeys job_keys(long long a, long long b) {
  JobKeys k;
  const unsigned long long ua = (unsigned long long)a, ub = (unsigned long long)b;
  k.k1 = a <= b ? ua : (KEY_TOP << 1) - ub;      // head by increasing a, then tail by decreasing b
  k.k2 = b <= a ? ub : (KEY_TOP << 1) - ua;      // head by increasing b, then tail by decreasing a
  k.k3 = ua;                                     // by increasing a
  k.k4 = KEY_TOP - ub;                           // by decreasing b
  return k;
}

__host__ __device__ inline size_t order_smem_bytes(int k_stride) {
  return (size_t)k_stride * (2 * sizeof(long long) + (ORDER_RULES - 1) * sizeof(short));
}

}  // namespace

__global__ void __launch_bounds__(32) order_kernel(int B, int k_stride, const long long* __restrict__ leg,
                                                   const long long* __restrict__ comp,
                                                   const int32_t* __restrict__ count,
                                                   const int32_t* __restrict__ eval_status,
                                                   int32_t* __restrict__ order, long long* __restrict__ best_ns,
                                                   long long* __restrict__ emission_ns, int32_t* __restrict__ rule,
                                                   int32_t* __restrict__ status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int b = blockIdx.x, lane = threadIdx.x;
  long long* a = reinterpret_cast<long long*>(smem_raw);
  long long* bt = a + k_stride;
  short* ord = reinterpret_cast<short*>(bt + k_stride);   // [rule - 1][position] -> job
  int32_t* ob = order + (size_t)b * k_stride;
  const int K = count[b];
  if (eval_status[b] != MOESCHED_ST_OK || K < 0 || K > k_stride) {
    for (int k = lane; k < k_stride; k += 32) ob[k] = -1;
    if (lane == 0) { best_ns[b] = 0; emission_ns[b] = 0; rule[b] = 0; status[b] = MOESCHED_ST_BAD_INPUT; }
    return;
  }
  for (int k = lane; k < K; k += 32) {
    a[k] = leg[(size_t)b * k_stride + k];
    bt[k] = comp[(size_t)b * k_stride + k];
  }
  __syncwarp();
  // rank of every job under each key: the number of jobs that come before it
  for (int k = lane; k < K; k += 32) {
    const JobKeys mine = job_keys(a[k], bt[k]);
    int r1 = 0, r2 = 0, r3 = 0, r4 = 0;
    for (int j = 0; j < K; ++j) {
      const JobKeys o = job_keys(a[j], bt[j]);
      const bool first = j < k;
      r1 += o.k1 < mine.k1 || (o.k1 == mine.k1 && first);
      r2 += o.k2 < mine.k2 || (o.k2 == mine.k2 && first);
      r3 += o.k3 < mine.k3 || (o.k3 == mine.k3 && first);
      r4 += o.k4 < mine.k4 || (o.k4 == mine.k4 && first);
    }
    ord[0 * k_stride + MS_AT(r1, K)] = (short)k;
    ord[1 * k_stride + MS_AT(r2, K)] = (short)k;
    // increasing a, placed alternately at the front and at the back
    ord[2 * k_stride + MS_AT((r3 & 1) ? K - 1 - (r3 >> 1) : (r3 >> 1), K)] = (short)k;
    ord[3 * k_stride + MS_AT(r4, K)] = (short)k;
  }
  __syncwarp();
  // one lane per candidate runs the three-stage recurrence on the fixed job times
  long long mk = 0x7fffffffffffffffLL;
  if (lane < ORDER_RULES) {
    long long dsp = 0, cmp = 0, cmb = 0;
    for (int p = 0; p < K; ++p) {
      const int k = lane == 0 ? p : MS_AT((int)ord[(lane - 1) * k_stride + p], K);
      dsp += a[k];
      cmp = max(dsp, cmp) + bt[k];
      cmb = max(cmp, cmb) + a[k];
    }
    mk = cmb;
  }
  const long long emission = __shfl_sync(FULL, mk, 0);
  long long best = mk;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(FULL, best, o));
  const int win = __ffs(__ballot_sync(FULL, mk == best)) - 1;   // the lower rule number on ties
  for (int p = lane; p < k_stride; p += 32) ob[p] = p < K ? (win == 0 ? p : (int)ord[(win - 1) * k_stride + p]) : -1;
  if (lane == 0) {
    best_ns[b] = best;
    emission_ns[b] = emission;
    rule[b] = win;
    status[b] = MOESCHED_ST_OK;
  }
}

// out[b][p] = in[b][order[b][p]] for the positions with an order entry >= 0; the others are left untouched.
__global__ void __launch_bounds__(256) permute_kernel(int B, int N, int k_stride, const uint8_t* __restrict__ perm,
                                                      const int32_t* __restrict__ dur,
                                                      const int32_t* __restrict__ order,
                                                      uint8_t* __restrict__ perm_out, int32_t* __restrict__ dur_out) {
  const long long slot = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // (b, position)
  const int lane = threadIdx.x & 31;
  if (slot >= (long long)B * k_stride) return;
  const int b = (int)(slot / k_stride), p = (int)(slot % k_stride);
  const int k = order[(size_t)b * k_stride + p];
  if (k < 0 || k >= k_stride) return;
  const uint8_t* src = perm + ((size_t)b * k_stride + k) * N;
  uint8_t* dst = perm_out + ((size_t)b * k_stride + p) * N;
  for (int i = lane; i < N; i += 32) dst[i] = src[i];
  if (lane == 0) dur_out[(size_t)b * k_stride + p] = dur[(size_t)b * k_stride + k];
}

// Number of matchings k in 1..count that minimises prefix_overlap[k-1] + price * prefix_unserved[k-1];
// the smallest such k on ties; 0 (and cost 0) for an empty or rejected schedule.
__global__ void __launch_bounds__(128) best_budget_kernel(int B, int k_stride, const int32_t* __restrict__ count,
                                                          const long long* __restrict__ prefix_overlap,
                                                          const long long* __restrict__ prefix_unserved,
                                                          long long price, int32_t* __restrict__ best_k,
                                                          long long* __restrict__ best_cost) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (b >= B) return;
  const int K = min(max(count[b], 0), k_stride);
  long long cost = 0x7fffffffffffffffLL;
  int at = 0x7fffffff, bad = 0;
  for (int k = lane; k < K; k += 32) {
    const long long o = prefix_overlap[(size_t)b * k_stride + k], u = prefix_unserved[(size_t)b * k_stride + k];
    if (o < 0 || u < 0) { bad = 1; continue; }
    const long long c = o + price * u;
    if (c < cost) { cost = c; at = k; }   // ascending k within the lane: the first minimum stays
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const long long oc = __shfl_xor_sync(FULL, cost, o);
    const int oa = __shfl_xor_sync(FULL, at, o);
    if (oc < cost || (oc == cost && oa < at)) { cost = oc; at = oa; }
  }
  bad = __any_sync(FULL, bad);
  if (lane == 0) {
    const bool none = bad || K == 0;
    best_k[b] = none ? 0 : at + 1;
    best_cost[b] = none ? 0 : cost;
  }
}

cudaError_t run_order(int B, int k_stride, const long long* leg, const long long* comp, const int32_t* count,
                      const int32_t* eval_status, int32_t* order, long long* best_ns, long long* emission_ns,
                      int32_t* rule, int32_t* status, cudaStream_t stream) {
  const size_t smem = order_smem_bytes(k_stride);
  cudaError_t e = cudaFuncSetAttribute(order_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  order_kernel<<<B, 32, smem, stream>>>(B, k_stride, leg, comp, count, eval_status, order, best_ns, emission_ns, rule,
                                        status);
  return cudaGetLastError();
}

cudaError_t run_permute(int B, int N, int k_stride, const uint8_t* perm, const int32_t* dur, const int32_t* order,
                        uint8_t* perm_out, int32_t* dur_out, cudaStream_t stream) {
  const long long slots = (long long)B * k_stride;
  const long long blocks = (slots + 7) / 8;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
  permute_kernel<<<(unsigned)blocks, 256, 0, stream>>>(B, N, k_stride, perm, dur, order, perm_out, dur_out);
  return cudaGetLastError();
}

cudaError_t run_best_budget(int B, int k_stride, const int32_t* count, const long long* prefix_overlap,
                            const long long* prefix_unserved, long long price, int32_t* best_k, long long* best_cost,
                            cudaStream_t stream) {
  best_budget_kernel<<<(B + 3) / 4, 128, 0, stream>>>(B, k_stride, count, prefix_overlap, prefix_unserved, price,
                                                      best_k, best_cost);
  return cudaGetLastError();
}

}  // namespace moesched
