// Schedule scoring (paper Sec. 4.1 "Execution time", Sec. 3.3), one warp per matrix.
//
// The demand matrix sits in shared memory and is consumed as the matchings are
// replayed; the schedule streams in from global memory. Matching k serves
// min(dur_k, remaining demand) tokens on each pair; the busiest pair drives the
// expert batch time; dispatch, compute and combine advance as a three-stage
// pipeline. Link idleness is obtained from totals: sum_k (N dur_k - s_k) equals
// N * sum_k dur_k minus all served tokens.
#include <type_traits>

#include "common.cuh"

namespace moesched {

__device__ __forceinline__ long long warp_sum64(long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
  return v;
}

// The stage recurrences x_k = max(a_k, x_{k-1}) + b_k are compositions of maps x -> max(x + p, q) (p = b_k,
// q = a_k + b_k), and such maps compose to a map of the same form: (p2, q2) after (p1, q1) is
// (p1 + p2, max(q1 + p2, q2)). An inclusive scan over the lanes (five steps) therefore gives every matching of a
// chunk its value at once, in exact integer arithmetic, instead of 32 dependent steps.
struct MaxPlus {
  long long p, q;
};
constexpr long long MAXPLUS_NONE = -(1LL << 62);   // q of the identity map (p = 0)
__device__ __forceinline__ MaxPlus maxplus_scan(MaxPlus m, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const long long up_p = __shfl_up_sync(FULL, m.p, o);
    const long long up_q = __shfl_up_sync(FULL, m.q, o);
    if (lane >= o) {   // the maps of the lower lanes act first
      m.q = max(up_q + m.p, m.q);
      m.p += up_p;
    }
  }
  return m;
}
__device__ __forceinline__ long long prefix_sum64(long long v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const long long up = __shfl_up_sync(FULL, v, o);
    if (lane >= o) v += up;
  }
  return v;
}

template <int CPL, typename View>
__device__ __forceinline__ long long matrix_sum(const View& M, int N, int lane, bool lane_in, int* any_negative) {
  long long acc = 0;
  int neg = 0;
  for (int r = 0; r < N; ++r) {
    if (lane_in) {
      RowVec<CPL> rv = load_cols<CPL>(M.row(r), lane);
#pragma unroll
      for (int s = 0; s < CPL; ++s)
        if (lane * CPL + s < N) { acc += rv.v[s]; neg |= rv.v[s] < 0; }
    }
  }
  if (any_negative) *any_negative = __any_sync(FULL, neg);
  return warp_sum64(acc);
}

// The lane's CPL destination bytes of one matching, packed little-endian.
template <int CPL>
struct Packed {
  typename std::conditional<(CPL > 4), unsigned long long, unsigned>::type v;
};
template <int CPL>
__device__ __forceinline__ Packed<CPL> load_dest(const uint8_t* row, int lane, int N, bool packed_ok) {
  Packed<CPL> p;
  const uint8_t* src = row + lane * CPL;
  if (packed_ok) {
    if constexpr (CPL == 1) p.v = *src;
    else if constexpr (CPL == 2) p.v = *reinterpret_cast<const unsigned short*>(src);
    else if constexpr (CPL == 4) p.v = *reinterpret_cast<const unsigned*>(src);
    else p.v = *reinterpret_cast<const unsigned long long*>(src);
  } else {
    p.v = 0;
#pragma unroll
    for (int s = 0; s < CPL; ++s)
      if (lane * CPL + s < N) p.v |= (decltype(p.v))src[s] << (8 * s);
  }
  return p;
}

// PREFIX: also write, after every matching k, the overlap makespan and the unserved tokens of the
// schedule cut after k+1 matchings (entries beyond count, or all entries of a bad schedule, are -1).
// JOBS (with PREFIX): the two per-matching arrays receive instead the job times of matching k in the
// three-stage flow shop: reconfiguration + transfer time, and the time of its expert batch.
// MODE 0: demand in this CTA's shared memory as int32; 1: split over a 2-CTA cluster; 2: held as
// 16-bit entries (matrices the pre-pass classified as narrow). only_class as in the greedy kernel.
template <int CPL, int MODE, bool PREFIX, bool JOBS = false>
__global__ void __launch_bounds__(128) eval_kernel(int B, int N, int S, const int32_t* __restrict__ demand, int k_stride,
                                                   const uint8_t* __restrict__ perm, const int32_t* __restrict__ dur,
                                                   const int32_t* __restrict__ count, moesched_model_t model,
                                                   FastDiv by_gbps, long long* __restrict__ overlap, long long* __restrict__ serial,
                                                   long long* __restrict__ idle_ns, long long* __restrict__ idle_tok,
                                                   long long* __restrict__ unserved, int32_t* status,
                                                   long long* __restrict__ prefix_overlap,
                                                   long long* __restrict__ prefix_unserved, int only_class) {
  constexpr int W = CPL;
  constexpr bool CLUSTER = MODE == 1;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  if (only_class != 0) {
    const int bb = CLUSTER ? (int)(blockIdx.x >> 1) : (int)(blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5));
    if (bb < B && status[bb] != only_class) return;
  }
  using View = typename std::conditional<MODE == 2, MatView16, MatView>::type;
  View D;
  int lane, b;
  bool loaded = true;
  if constexpr (MODE == 2) {
    WarpCtx16 cx = warp_prologue16<CPL, true>(B, N, S, demand, smem_raw);
    if (!cx.worker) return;
    lane = cx.lane; b = cx.b; D = cx.M; loaded = cx.loaded;
  } else {
    WarpCtx cx = warp_prologue<CPL, CLUSTER>(B, N, S, demand, smem_raw);
    if (!cx.worker) { cluster_epilogue<CLUSTER>(); return; }
    lane = cx.lane; b = cx.b; D = cx.M; loaded = cx.loaded;
  }
  const bool lane_in = lane * CPL < S;

  int bad = loaded ? 0 : 1;
  int neg = 0;
  const long long total = matrix_sum<CPL, View>(D, N, lane, lane_in, &neg);
  bad |= neg;
  const int K = count[b];
  if (K < 0 || K > k_stride) bad = 1;

  long long dsp = 0, cmp = 0, cmb = 0, ser = 0, comp_sum = 0, dsp1 = 0, dur_sum = 0, served_sum = 0;
  const uint8_t* pb = perm + (size_t)b * k_stride * N;
  const int32_t* db = dur + (size_t)b * k_stride;

  unsigned allcols[W];   // the set of all N columns
#pragma unroll
  for (int w = 0; w < W; ++w) allcols[w] = ~ge_word(N, w);
  if (!bad) {
    // one aligned word holds the lane's CPL destinations when rows of the schedule are CPL-aligned
    const bool packed_ok = (N % CPL == 0) && ((reinterpret_cast<uintptr_t>(pb) & (CPL - 1)) == 0);
    for (int k0 = 0; k0 < K && !bad; k0 += 32) {
      // lane q prepares the transfer time of matching k0+q
      const int kk = k0 + lane;
      const int dk_mine = kk < K ? db[kk] : 0;
      if (__any_sync(FULL, dk_mine < 0)) { bad = 1; break; }
      // dk < 2^31, bytes_per_token and link_gbps <= 2^20: the dividend stays below 2^55
      const long long t_mine =
          fast_div((long long)dk_mine * model.bytes_per_token * 8 + model.link_gbps - 1, by_gbps);
      const int kend = min(32, K - k0);
      // fetch the lane's destinations of all matchings of the chunk before using any of them:
      // 32 independent loads in flight instead of one dependent load per matching
      Packed<CPL> dest[32];
#pragma unroll
      for (int q = 0; q < 32; ++q) {
        dest[q].v = 0;
        if (q < kend && lane * CPL < N) dest[q] = load_dest<CPL>(pb + (size_t)(k0 + q) * N, lane, N, packed_ok);
      }
      // replay: lane q keeps what matching k0+q served (largest pair, total)
      int g_mine = 0;
      long long served_mine = 0;
#pragma unroll
      for (int q = 0; q < 32; ++q) {
        if (q < kend && !bad) {
          const int dk = __shfl_sync(FULL, dk_mine, q);
          unsigned cols[W];
#pragma unroll
          for (int w = 0; w < W; ++w) cols[w] = 0u;
          int g = 0, oob = 0;
          unsigned slo = 0u, shi = 0u;   // served tokens of this matching, low and high halves
#pragma unroll
          for (int s = 0; s < CPL; ++s) {
            const int r = lane * CPL + s;
            if (r < N) {
              const int j = (int)((dest[q].v >> (8 * s)) & 0xff);
              if (j < N) {
                set_bit<W>(cols, j);
                auto* p = D.row(r) + MS_AT(j, N);
                const int val = *p;
                const int sv = min(dk, val);
                *p = val - sv;
                g = max(g, sv);
                if constexpr (PREFIX) { slo += (unsigned)sv & 0xffffu; shi += (unsigned)sv >> 16; }
              } else {
                oob = 1;
              }
            }
          }
          // N destinations, none out of range: a permutation iff every column 0..N-1 is hit
          unsigned missing = 0u;
#pragma unroll
          for (int w = 0; w < W; ++w) missing |= ~__reduce_or_sync(FULL, cols[w]) & allcols[w];
          if (__any_sync(FULL, oob) || missing != 0u) {
            bad = 1;
          } else {
            g = __reduce_max_sync(FULL, g);
            if (lane == q) g_mine = g;
            if constexpr (PREFIX) {
              const long long sv_all = ((long long)__reduce_add_sync(FULL, shi) << 16) + __reduce_add_sync(FULL, slo);
              if (lane == q) served_mine = sv_all;
            }
          }
          // (no barrier here: a lane only ever touches the rows it owns; the sums after the loop have their own)
        }
      }
      if (bad) break;
      // times of the chunk, one matching per lane, then the three-stage recurrence in order
      const bool mine = lane < kend;
      const long long comp_mine = mine ? batch_time_ns(model, g_mine) : 0;
      const long long leg_mine = mine ? model.reconfig_ns + t_mine : 0;
      ser += warp_sum64(2 * leg_mine + comp_mine);
      comp_sum += warp_sum64(comp_mine);
      dur_sum += warp_sum64((long long)dk_mine);
      // stage sums beyond 2^60 ns are out of range (a chunk adds less than 2^61, so nothing has wrapped yet)
      if (ser - comp_sum > (2LL << 60) || comp_sum > (1LL << 60)) { bad = 1; break; }
      // lane q gets the three stage times after matching k0+q; lanes beyond the chunk carry identity maps
      const long long dsp_mine = dsp + prefix_sum64(leg_mine, lane);
      MaxPlus f;
      f.p = comp_mine;
      f.q = mine ? dsp_mine + comp_mine : MAXPLUS_NONE;
      f = maxplus_scan(f, lane);
      const long long cmp_mine = max(cmp + f.p, f.q);
      MaxPlus h;
      h.p = leg_mine;
      h.q = mine ? cmp_mine + leg_mine : MAXPLUS_NONE;
      h = maxplus_scan(h, lane);
      const long long cmb_mine = max(cmb + h.p, h.q);
      if (k0 == 0) dsp1 = __shfl_sync(FULL, dsp_mine, 0);
      dsp = __shfl_sync(FULL, dsp_mine, kend - 1);
      cmp = __shfl_sync(FULL, cmp_mine, kend - 1);
      cmb = __shfl_sync(FULL, cmb_mine, kend - 1);
      if constexpr (PREFIX) {
        const long long run = prefix_sum64(served_mine, lane);   // inclusive prefix sum over the lanes
        if (mine) {
          prefix_overlap[(size_t)b * k_stride + k0 + lane] = JOBS ? leg_mine : cmb_mine;
          prefix_unserved[(size_t)b * k_stride + k0 + lane] = JOBS ? comp_mine : total - (served_sum + run);
        }
        served_sum += __shfl_sync(FULL, run, 31);
      }
    }
    if (dur_sum > (1LL << 40)) bad = 1;
  }

  long long left = 0;
  if (!bad) {
    __syncwarp();
    left = matrix_sum<CPL, View>(D, N, lane, lane_in, nullptr);
  }
  if constexpr (PREFIX) {
    const int from = bad ? 0 : K;
    for (int k = from + lane; k < k_stride; k += 32) {
      prefix_overlap[(size_t)b * k_stride + k] = -1;
      prefix_unserved[(size_t)b * k_stride + k] = -1;
    }
  }
  if (lane == 0) {
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
  cluster_epilogue<CLUSTER>();
}

template <int MODE>
static cudaError_t launch_eval_mode(const Geometry& ge, int B, int N, const int32_t* demand, int k_stride,
                                    const uint8_t* perm, const int32_t* dur, const int32_t* count,
                                    const moesched_model_t& model, long long* overlap, long long* serial,
                                    long long* idle_ns, long long* idle_tok, long long* unserved, int32_t* status,
                                    long long* prefix_overlap, long long* prefix_unserved, int only_class,
                                    bool jobs, cudaStream_t stream) {
  const bool prefix = prefix_overlap != nullptr;
  const FastDiv by_gbps = make_fastdiv(model.link_gbps);
#define MOESCHED_GO(C)                                                                                             \
  do {                                                                                                             \
    if (prefix && jobs)                                                                                            \
      return launch_warp_kernel(eval_kernel<C, MODE, true, true>, ge, B, stream, B, N, ge.S, demand, k_stride,     \
                                perm, dur, count, model, by_gbps, overlap, serial, idle_ns, idle_tok, unserved,   \
                                status, prefix_overlap, prefix_unserved, only_class);                              \
    if (prefix)                                                                                                    \
      return launch_warp_kernel(eval_kernel<C, MODE, true>, ge, B, stream, B, N, ge.S, demand, k_stride, perm,     \
                                dur, count, model, by_gbps, overlap, serial, idle_ns, idle_tok, unserved,         \
                                status, prefix_overlap, prefix_unserved, only_class);                              \
    return launch_warp_kernel(eval_kernel<C, MODE, false>, ge, B, stream, B, N, ge.S, demand, k_stride, perm, dur, \
                              count, model, by_gbps, overlap, serial, idle_ns, idle_tok, unserved, status,        \
                              prefix_overlap, prefix_unserved, only_class);                                        \
  } while (0)
  switch (ge.cpl) {
    case 1: MOESCHED_GO(1);
    case 2: MOESCHED_GO(2);
    case 4: MOESCHED_GO(4);
    default: MOESCHED_GO(8);
  }
#undef MOESCHED_GO
}

cudaError_t run_eval(int B, int N, const int32_t* demand, int k_stride, const uint8_t* perm, const int32_t* dur,
                     const int32_t* count, const moesched_model_t& model, long long* overlap, long long* serial,
                     long long* idle_ns, long long* idle_tok, long long* unserved, int32_t* status,
                     long long* prefix_overlap, long long* prefix_unserved, cudaStream_t stream, bool jobs) {
  const Geometry ge = plan_geometry(N);
  int only_class = 0;
  if (N >= 48) {
    // as in the greedy path: narrow matrices first, in the 16-bit layout, then the rest
    cudaError_t e = classify_matrices(B, N, demand, status, stream);
    if (e != cudaSuccess) return e;
    if (N > 128 && B < 8 * sm_count() && prefix_overlap == nullptr && k_stride <= 65535 * 32) {
      // few large matrices: one CTA per matrix instead of one warp (N = 256, B = 256 on a BvN schedule:
      // 33 ms against 74 ms; at N = 128, B = 1024 one warp per matrix is the faster, 17 ms against 20 ms)
      e = run_eval_team(B, N, demand, k_stride, perm, dur, count, model, overlap, serial, idle_ns, idle_tok, unserved,
                        status, stream);
    } else {
      Geometry g16 = ge;
      g16.cluster = false;
      g16.wpb = 1;
      g16.smem = warp_smem_bytes16(N, g16.S, g16.cpl);
      e = launch_eval_mode<2>(g16, B, N, demand, k_stride, perm, dur, count, model, overlap, serial, idle_ns,
                              idle_tok, unserved, status, prefix_overlap, prefix_unserved, CLASS_U16, jobs, stream);
    }
    if (e != cudaSuccess) return e;
    only_class = CLASS_I32;
  }
  if (ge.cluster)
    return launch_eval_mode<1>(ge, B, N, demand, k_stride, perm, dur, count, model, overlap, serial, idle_ns,
                               idle_tok, unserved, status, prefix_overlap, prefix_unserved, only_class, jobs, stream);
  return launch_eval_mode<0>(ge, B, N, demand, k_stride, perm, dur, count, model, overlap, serial, idle_ns, idle_tok,
                             unserved, status, prefix_overlap, prefix_unserved, only_class, jobs, stream);
}

}  // namespace moesched
