// Schedule scoring (paper Sec. 4.1 "Execution time", Sec. 3.3) with one CTA per matrix, for the
// large, small-batch case in which one warp per matrix leaves most of the machine idle (N > 128 and
// fewer than 8 matrices per SM). Same results as eval_kernel.cu. Thread t owns row t of the demand,
// held as 16-bit entries in shared memory (the kernel takes the matrices the class pre-pass marked
// narrow; the others stay with the one-warp kernels). The schedule is consumed 32 matchings at a
// time: every thread fetches its destination in each of them, the 32 permutation checks and the
// replay need no exchange between threads beyond a per-matching maximum, and warp 0 then runs the
// times and the three-stage recurrence of the chunk exactly as the one-warp kernel does.
#include "common.cuh"

namespace moesched {

namespace {

struct EvalTeamState {
  int gmax[32];        // largest served pair of each matching of the chunk
  int dur[32];         // its duration
  int flags[4];        // 0: chunk is bad, 1: a sum left its range
  long long sums[4];   // block reductions: total demand, leftover
};

__host__ __device__ inline size_t eval_team_smem(int N) {
  return align16((size_t)N * N * 2) + align16((size_t)32 * N * 2) + sizeof(EvalTeamState);
}

__device__ __forceinline__ long long block_sum64(long long v, long long* slot, int lane) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
  if (lane == 0 && v != 0) atomicAdd(reinterpret_cast<unsigned long long*>(slot), (unsigned long long)v);
  __syncthreads();
  return *slot;
}

}  // namespace

template <int NW>
__global__ void __launch_bounds__(32 * NW) eval_team_kernel(int B, int N, const int32_t* __restrict__ demand,
                                                            int k_stride, const uint8_t* __restrict__ perm,
                                                            const int32_t* __restrict__ dur,
                                                            const int32_t* __restrict__ count, moesched_model_t model,
                                                            FastDiv by_gbps, long long* __restrict__ overlap,
                                                            long long* __restrict__ serial,
                                                            long long* __restrict__ idle_ns,
                                                            long long* __restrict__ idle_tok,
                                                            long long* __restrict__ unserved, int32_t* status) {
  constexpr int NT = 32 * NW;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int b = blockIdx.x;
  if (status[b] != CLASS_U16) return;   // uniform: wide matrices are scored by the one-warp kernels
  unsigned short* D = reinterpret_cast<unsigned short*>(smem_raw);
  unsigned short* marks = reinterpret_cast<unsigned short*>(smem_raw + align16((size_t)N * N * 2));
  EvalTeamState* st =
      reinterpret_cast<EvalTeamState*>(smem_raw + align16((size_t)N * N * 2) + align16((size_t)32 * N * 2));
  const bool in = t < N;

  // demand into shared memory (the class pre-pass guarantees 0 <= entry <= 65535), total, marks cleared
  const int32_t* src = demand + (size_t)b * N * N;
  long long mine = 0;
  for (int e = t; e < N * N; e += NT) {
    const int v = src[e];
    D[e] = (unsigned short)v;
    mine += v;
  }
  for (int e = t; e < 32 * N; e += NT) marks[e] = 0;
  if (t < 4) { st->sums[t] = 0; st->flags[t] = 0; }
  __syncthreads();
  const long long total = block_sum64(mine, &st->sums[0], lane);

  const int K = count[b];
  bool bad = K < 0 || K > k_stride;
  long long dsp = 0, cmp = 0, cmb = 0, ser = 0, comp_sum = 0, dsp1 = 0, dur_sum = 0;   // live in warp 0
  const uint8_t* pb = perm + (size_t)b * k_stride * N;
  const int32_t* db = dur + (size_t)b * k_stride;
  unsigned short* myrow = D + (size_t)t * N;

  for (int k0 = 0, chunk = 1; !bad && k0 < K; k0 += 32, ++chunk) {
    const int kend = min(32, K - k0);
    const unsigned short stamp = (unsigned short)chunk;   // the launcher admits at most 65535 chunks: never 0, never repeats
    if (t < 32) {
      const int dk = t < kend ? db[k0 + t] : 0;
      st->dur[t] = dk;
      st->gmax[t] = 0;
      if (dk < 0) st->flags[0] = 1;
    }
    // destinations of row t in the chunk's matchings; each marks its column
    int dest[32];
    int oob = 0;
#pragma unroll
    for (int q = 0; q < 32; ++q) {
      dest[q] = 0;
      if (q < kend && in) {
        const int j = pb[(size_t)(k0 + q) * N + t];
        dest[q] = j;
        if (j < N) marks[q * N + j] = stamp;
        else oob = 1;
      }
    }
    if (oob) st->flags[0] = 1;
    __syncthreads();
    // a matching is a permutation iff every column was marked (N marks, none out of range)
    {
      int missing = 0;
#pragma unroll
      for (int q = 0; q < 32; ++q)
        if (q < kend && in) missing |= marks[q * N + t] != stamp;
      if (missing) st->flags[0] = 1;
    }
    __syncthreads();
    if (st->flags[0]) { bad = true; break; }
    // replay: only the owner touches row t; the largest served pair of each matching is collected
#pragma unroll
    for (int q = 0; q < 32; ++q) {
      if (q < kend) {
        int sv = 0;
        if (in) {
          const int dk = st->dur[q];
          const int val = myrow[MS_AT(dest[q], N)];
          sv = min(dk, val);
          myrow[MS_AT(dest[q], N)] = (unsigned short)(val - sv);
        }
        const int g = __reduce_max_sync(FULL, sv);
        if (lane == 0 && g > 0) atomicMax(&st->gmax[q], g);
      }
    }
    __syncthreads();
    // times of the chunk, one matching per lane of warp 0, then the three-stage recurrence in order
    if (warp == 0) {
      const bool has = lane < kend;
      const int dk_mine = has ? st->dur[lane] : 0;
      const int g_mine = has ? st->gmax[lane] : 0;
      const long long t_mine =
          fast_div((long long)dk_mine * model.bytes_per_token * 8 + model.link_gbps - 1, by_gbps);
      const long long comp_mine = has ? batch_time_ns(model, g_mine) : 0;
      const long long leg_mine = has ? model.reconfig_ns + t_mine : 0;
      long long a = 2 * leg_mine + comp_mine, c = comp_mine, d = (long long)dk_mine;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_xor_sync(FULL, a, o);
        c += __shfl_xor_sync(FULL, c, o);
        d += __shfl_xor_sync(FULL, d, o);
      }
      ser += a;
      comp_sum += c;
      dur_sum += d;
      // stage sums beyond 2^60 ns are out of range (a chunk adds less than 2^61, so nothing has wrapped yet)
      if (lane == 0 && (ser - comp_sum > (2LL << 60) || comp_sum > (1LL << 60))) st->flags[1] = 1;
      for (int q = 0; q < kend; ++q) {
        const long long leg = __shfl_sync(FULL, leg_mine, q);
        const long long comp = __shfl_sync(FULL, comp_mine, q);
        dsp += leg;
        if (k0 + q == 0) dsp1 = dsp;
        cmp = max(dsp, cmp) + comp;
        cmb = max(cmp, cmb) + leg;
      }
    }
    __syncthreads();
    if (st->flags[1]) { bad = true; break; }
  }
  if (warp == 0 && lane == 0 && dur_sum > (1LL << 40)) st->flags[1] = 1;
  __syncthreads();
  if (st->flags[1]) bad = true;

  // demand left over
  long long left = 0;
  if (!bad) {
    long long part = 0;
    for (int e = t; e < N * N; e += NT) part += D[e];
    left = block_sum64(part, &st->sums[1], lane);
  }
  if (t == 0) {
    if (bad) {
      overlap[b] = serial[b] = idle_ns[b] = idle_tok[b] = unserved[b] = 0;
      status[b] = MOESCHED_ST_BAD_INPUT;
    } else {
      overlap[b] = cmb;
      serial[b] = ser;
      idle_ns[b] = K > 0 ? (cmp - dsp1) - comp_sum : 0;
      idle_tok[b] = (long long)N * dur_sum - (total - left);
      unserved[b] = left;
      status[b] = MOESCHED_ST_OK;
    }
  }
}

// ---- host side ---------------------------------------------------------------------------

// Scores the matrices whose status holds CLASS_U16 (the others are left for the one-warp kernels).
cudaError_t run_eval_team(int B, int N, const int32_t* demand, int k_stride, const uint8_t* perm, const int32_t* dur,
                          const int32_t* count, const moesched_model_t& model, long long* overlap, long long* serial,
                          long long* idle_ns, long long* idle_tok, long long* unserved, int32_t* status,
                          cudaStream_t stream) {
  const size_t smem = eval_team_smem(N);
  const FastDiv by_gbps = make_fastdiv(model.link_gbps);
  cudaError_t e;
  if (N <= 128) {
    e = cudaFuncSetAttribute(eval_team_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    eval_team_kernel<4><<<B, 128, smem, stream>>>(B, N, demand, k_stride, perm, dur, count, model, by_gbps, overlap,
                                                  serial, idle_ns, idle_tok, unserved, status);
  } else {
    e = cudaFuncSetAttribute(eval_team_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    eval_team_kernel<8><<<B, 256, smem, stream>>>(B, N, demand, k_stride, perm, dur, count, model, by_gbps, overlap,
                                                  serial, idle_ns, idle_tok, unserved, status);
  }
  return cudaGetLastError();
}

}  // namespace moesched
