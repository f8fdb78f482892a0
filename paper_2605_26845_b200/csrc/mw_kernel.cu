// Greedy max-weight decomposition (paper Sec. 3.2), one warp per demand matrix.
//
// Each greedy step solves one assignment problem on the residual matrix R by
// shortest augmenting paths on cost = -R (a Jonker-Volgenant style search that
// keeps only the column duals v, warm-started from the previous step), derives
// the row duals, marks the tight edges and hands that graph to canonicalise(),
// which returns the lexicographically smallest optimal permutation. The matched
// entries are then served whole; the largest one is the matching's duration.
#include <type_traits>

#include "common.cuh"

namespace moesched {

template <int CPL>
struct MwState {
  int v[CPL];     // column duals of the cost problem
  Match<CPL> M;   // row assigned to each of the lane's columns
};

// Tight edges under the column duals v: T[s] = rows whose smallest reduced cost (cost - v over the
// row) is attained in the lane's column s.
template <int CPL, typename View>
__device__ __forceinline__ void tight_graph(const View& R, int N, int lane, bool lane_in, const int (&v)[CPL],
                                            unsigned (&T)[CPL][CPL]) {
  constexpr int W = CPL;
#pragma unroll
  for (int s = 0; s < CPL; ++s)
#pragma unroll
    for (int w = 0; w < W; ++w) T[s][w] = 0u;
#pragma unroll
  for (int w = 0; w < W; ++w) {
    for (int q = 0; q < 32; ++q) {
      const int r = w * 32 + q;
      if (r >= N) break;
      RowVec<CPL> rv;
      if (lane_in) rv = load_cols<CPL>(R.row(r), lane);
      int red[CPL], lm = INF32;
#pragma unroll
      for (int s = 0; s < CPL; ++s) {
        red[s] = (lane * CPL + s < N) ? -rv.v[s] - v[s] : INF32;
        lm = min(lm, red[s]);
      }
      const int u = __reduce_min_sync(FULL, lm);
#pragma unroll
      for (int s = 0; s < CPL; ++s)
        if (red[s] == u && lane * CPL + s < N) T[s][w] |= 1u << q;
    }
  }
}

// One assignment problem. The column duals v carry over from the previous greedy step
// (weights only decreased, so they are still feasible); they are shifted so that the largest
// is zero, which keeps every intermediate value within a few multiples of the largest entry.
// Each row first tries the column that minimises cost - v (lowest column on ties) and keeps
// it if that column is still free: such a row is matched along a tight edge. When at least half
// of the rows are left over (sparse, tie-rich residuals), each of them is first offered an
// augmenting path of tight edges, which matches it without touching the duals (measured on the
// N = 256 configuration: 2.4 k instead of 13 k column scans per matching; with fewer rows left
// over the searches cost more than they save). The remaining rows are added one by one by a
// shortest-augmenting-path search that settles one column per scan and updates only the column
// duals. Returns false if an iteration limit was hit.
template <int CPL, typename View>
__device__ __forceinline__ bool solve_assignment(const View& R, int N, int lane, bool lane_in,
                                                 MwState<CPL>& st, short* x, unsigned (&work)[MOESCHED_WORK_FIELDS]) {
  constexpr int W = CPL;
  bool ok = true;
  {
    int vmax = -INF32;
#pragma unroll
    for (int s = 0; s < CPL; ++s)
      if (lane * CPL + s < N) vmax = max(vmax, st.v[s]);
    vmax = __reduce_max_sync(FULL, vmax);
#pragma unroll
    for (int s = 0; s < CPL; ++s) st.v[s] -= vmax;
    st.M.reset();
  }
  for (int r = lane; r < N; r += 32) x[r] = -1;
  unsigned freerows[W];
#pragma unroll
  for (int w = 0; w < W; ++w) freerows[w] = 0u;
  __syncwarp();
  for (int r = 0; r < N; ++r) {
    RowVec<CPL> rv;
    if (lane_in) rv = load_cols<CPL>(R.row(r), lane);
    int lmin = INF32, lslot = 0;
#pragma unroll
    for (int ss = 0; ss < CPL; ++ss) {
      const int s = CPL - 1 - ss;
      const int d = (lane * CPL + s < N) ? -rv.v[s] - st.v[s] : INF32;
      if (d <= lmin) { lmin = d; lslot = s; }
    }
    const int u = __reduce_min_sync(FULL, lmin);
    const unsigned ball = __ballot_sync(FULL, lmin == u);
    const int L = __ffs(ball) - 1;
    const int sl = __shfl_sync(FULL, lslot, L);
    const int owner = __shfl_sync(FULL, st.M.row_of(sl), L);
    if (owner < 0) {
      if (lane == L) st.M.assign(sl, r);
      x[r] = (short)(L * CPL + sl);   // every lane: a lane later reads what it wrote itself (see hist_store)
    } else {
      set_bit<W>(freerows, r);
    }
    work[WK_TIGHT]++;
  }
  __syncwarp();
  {
    int nfree = 0;
#pragma unroll
    for (int w = 0; w < W; ++w) nfree += __popc(freerows[w]);
    if (2 * nfree >= N) {
      unsigned T[CPL][CPL];
      tight_graph<CPL, View>(R, N, lane, lane_in, st.v, T);
      unsigned left[W];
#pragma unroll
      for (int w = 0; w < W; ++w) { left[w] = freerows[w]; freerows[w] = 0u; }
      unsigned search_work[MOESCHED_WORK_FIELDS], moved[W];   // not reported: the search's own counters
      int lo = 0, hi = 0;
      for (int it = 0; it < N; ++it) {
        const int f = lowest_bit<W>(left);
        if (f < 0) break;
        clear_bit<W>(left, f);
        if (augment_from<CPL>(N, lane, f, T, st.M, x, lo, hi, moved, search_work)) work[WK_SKIP]++;
        else set_bit<W>(freerows, f);
      }
      __syncwarp();
    }
  }
  for (int outer = 0; outer < N; ++outer) {
    const int f = lowest_bit<W>(freerows);
    if (f < 0) break;
    clear_bit<W>(freerows, f);
    int dist[CPL], pred[CPL];
    unsigned scanned = 0u;     // bit s: the lane's column s is settled
    {
      RowVec<CPL> rv;
      if (lane_in) rv = load_cols<CPL>(R.row(MS_AT(f, N)), lane);
#pragma unroll
      for (int s = 0; s < CPL; ++s) {
        bool valid = lane * CPL + s < N;
        dist[s] = valid ? -rv.v[s] - st.v[s] : INF32;
        pred[s] = f;
        if (!valid) scanned |= 1u << s;
      }
    }
    int jfin = -1, mu = 0;
    for (int it = 0; it < N; ++it) {
      int lmin = INF32, lslot = 0;
#pragma unroll
      for (int ss = 0; ss < CPL; ++ss) {
        const int s = CPL - 1 - ss;
        int d = ((scanned >> s) & 1u) ? INF32 : dist[s];
        if (d <= lmin) { lmin = d; lslot = s; }
      }
      mu = __reduce_min_sync(FULL, lmin);
      const unsigned ball = __ballot_sync(FULL, lmin == mu);
      const int L = __ffs(ball) - 1;
      const int sl = __shfl_sync(FULL, lslot, L);
      if (lane == L) scanned |= 1u << sl;
      const int i = __shfl_sync(FULL, st.M.row_of(sl), L);
      work[WK_SCAN]++;
      if (i < 0) { jfin = L * CPL + sl; break; }
      RowVec<CPL> rv;
      if (lane_in) rv = load_cols<CPL>(R.row(MS_AT(i, N)), lane);
      // the owner of the settled column forms h from its own entry and dual: one broadcast instead of two
      const int h = __shfl_sync(FULL, -pick<CPL>(rv.v, sl) - pick<CPL>(st.v, sl) - mu, L);
#pragma unroll
      for (int s = 0; s < CPL; ++s) {
        int nd = -rv.v[s] - st.v[s] - h;
        if (!((scanned >> s) & 1u) && nd < dist[s]) { dist[s] = nd; pred[s] = i; }
      }
    }
    if (jfin < 0) { ok = false; break; }
    // settled columns move their dual so that the new shortest-path tree stays tight
#pragma unroll
    for (int s = 0; s < CPL; ++s)
      if (((scanned >> s) & 1u) && lane * CPL + s < N) st.v[s] += dist[s] - mu;
    // flip the path back to row f
    int j = jfin;
    for (int it = 0; it <= N; ++it) {
      const int L = j / CPL, sl = j % CPL;
      const int i = __shfl_sync(FULL, pick<CPL>(pred, sl), L);
      const int jprev = x[MS_AT(i, N)];
      if (lane == L) st.M.assign(sl, i);
      x[MS_AT(i, N)] = (short)j;   // every lane
      if (i == f) break;
      j = jprev;
      if (j < 0) { ok = false; break; }
    }
    work[WK_AUG]++;
  }
  if (any_bit<W>(freerows)) ok = false;
  return ok;
}

// Matrices are sorted into two classes by a streaming pre-pass that leaves the class in status[b]:
// all entries within 16 bits (held as 16-bit values: twice as many matrices per SM) or not.
__global__ void __launch_bounds__(256) mw_classify_kernel(int B, int N, const int32_t* __restrict__ demand,
                                                          int32_t* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (b >= B) return;
  const int32_t* D = demand + (size_t)b * N * N;
  int wide = 0;
  for (int e = lane; e < N * N; e += 32) wide |= (unsigned)D[e] > 65535u;   // negative entries count as wide
  wide = __any_sync(FULL, wide);
  if (lane == 0) status[b] = wide ? CLASS_I32 : CLASS_U16;
}

// MODE 0: matrix in this CTA's shared memory as int32; 1: split over a 2-CTA cluster; 2: 16-bit entries.
// only_class != 0: handle only the matrices whose status[b] holds that class.
// COUNT: the per-matrix work counters are wanted (register increments the compiler drops otherwise).
template <int CPL, int MODE, bool COUNT>
__global__ void __launch_bounds__(128) mw_kernel(int B, int N, int S, const int32_t* __restrict__ demand, int k_max,
                                                 uint8_t* __restrict__ perm, int32_t* __restrict__ dur,
                                                 int32_t* __restrict__ count, int32_t* __restrict__ residual,
                                                 int32_t* status, long long* __restrict__ work_out, int only_class) {
  constexpr bool CLUSTER = MODE == 1;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  if (only_class != 0) {
    const int bb = CLUSTER ? (int)(blockIdx.x >> 1) : (int)(blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5));
    if (bb < B && status[bb] != only_class) return;   // both CTAs of a cluster see the same class
  }
  using View = typename std::conditional<MODE == 2, MatView16, MatView>::type;
  View R;
  int lane, b;
  short* x;
  unsigned* hist;
  bool loaded = true;
  if constexpr (MODE == 2) {
    WarpCtx16 cx = warp_prologue16<CPL, false>(B, N, S, demand, smem_raw);
    if (!cx.worker) return;
    lane = cx.lane; b = cx.b; R = cx.M; x = cx.x; hist = cx.hist; loaded = cx.loaded;
  } else {
    WarpCtx cx = warp_prologue<CPL, CLUSTER>(B, N, S, demand, smem_raw);
    if (!cx.worker) { cluster_epilogue<CLUSTER>(); return; }
    lane = cx.lane; b = cx.b; R = cx.M; x = cx.x; hist = cx.hist; loaded = cx.loaded;
  }

  unsigned work[MOESCHED_WORK_FIELDS];
#pragma unroll
  for (int q = 0; q < MOESCHED_WORK_FIELDS; ++q) work[q] = 0u;

  const bool lane_in = lane * CPL < S;
  int st_code = MOESCHED_ST_OK;
  int k = 0;

  // validate, find the largest entry, count the non-zero entries
  int nnz = 0;
  {
    int mx = 0, neg = 0, cnt = 0;
    for (int r = 0; r < N; ++r) {
      if (lane_in) {
        RowVec<CPL> rv = load_cols<CPL>(R.row(r), lane);
#pragma unroll
        for (int s = 0; s < CPL; ++s) {
          if (lane * CPL + s < N) {
            neg |= rv.v[s] < 0;
            mx = max(mx, rv.v[s]);
            cnt += rv.v[s] != 0;
          }
        }
      }
    }
    neg = __any_sync(FULL, neg);
    mx = __reduce_max_sync(FULL, mx);
    nnz = __reduce_add_sync(FULL, cnt);
    if (neg || mx > MOESCHED_MW_MAX_ENTRY) st_code = MOESCHED_ST_BAD_INPUT;
    if (!loaded) st_code = MOESCHED_ST_INTERNAL;
  }

  if (st_code == MOESCHED_ST_OK) {
    MwState<CPL> st;
#pragma unroll
    for (int s = 0; s < CPL; ++s) st.v[s] = 0;
    st.M.reset();
    uint8_t* pout = perm + (size_t)b * k_max * N;
    int32_t* dout = dur + (size_t)b * k_max;
    while (k < k_max && nnz > 0) {
      if (!solve_assignment<CPL, View>(R, N, lane, lane_in, st, x, work)) { st_code = MOESCHED_ST_INTERNAL; break; }
      // tight edges: row r is tight to column c iff cost(r,c) - v[c] equals the row minimum
      unsigned C[CPL][CPL];
      tight_graph<CPL, View>(R, N, lane, lane_in, st.v, C);
      CanonMemo<CPL> memo;   // unused: every greedy step has a new graph
      memo.reset();
      if (!canonicalise<CPL, false>(N, lane, 0, N - 1, C, st.M, x, hist, memo, work)) {
        st_code = MOESCHED_ST_INTERNAL;
        break;
      }
      // serve: the heaviest matched pair sets the duration; matched entries are sent whole
      int dmax = 0, served = 0;
#pragma unroll
      for (int s = 0; s < CPL; ++s) {
        const int c = lane * CPL + s;
        if (c < N && st.M.mr[s] >= 0) {
          auto* p = R.row(MS_AT(st.M.mr[s], N)) + c;
          const int val = *p;
          dmax = max(dmax, val);
          served += val != 0;
          *p = 0;
        }
      }
      dmax = __reduce_max_sync(FULL, dmax);
      nnz -= __reduce_add_sync(FULL, served);
      __syncwarp();
      for (int r = lane; r < N; r += 32) pout[(size_t)k * N + r] = (uint8_t)x[r];
      if (lane == 0) dout[k] = dmax;
      ++k;
      work[WK_MATCH]++;
    }
    if (st_code == MOESCHED_ST_OK && nnz > 0) st_code = MOESCHED_ST_TRUNCATED;
  }

  if (st_code == MOESCHED_ST_BAD_INPUT) k = 0;
  if (lane == 0) {
    count[b] = k;
    status[b] = st_code;
  }
  if (residual != nullptr && st_code != MOESCHED_ST_BAD_INPUT) {
    int32_t* ro = residual + (size_t)b * N * N;
    for (int r = 0; r < N; ++r) {
      const auto* rp = R.row(r);
      for (int c = lane; c < N; c += 32) ro[(size_t)r * N + c] = rp[c];
    }
  }
  if constexpr (COUNT) {
    if (work_out != nullptr && lane == 0) {
#pragma unroll
      for (int q = 0; q < MOESCHED_WORK_FIELDS; ++q) work_out[(size_t)b * MOESCHED_WORK_FIELDS + q] = work[q];
    }
  }
  cluster_epilogue<CLUSTER>();
}

cudaError_t classify_matrices(int B, int N, const int32_t* demand, int32_t* status, cudaStream_t stream) {
  mw_classify_kernel<<<(B + 7) / 8, 256, 0, stream>>>(B, N, demand, status);
  return cudaGetLastError();
}

// ---- host side ---------------------------------------------------------------------------

template <int MODE>
static cudaError_t launch_mw_mode(Geometry ge, int B, int N, const int32_t* demand, int k_max, uint8_t* perm,
                                  int32_t* dur, int32_t* count, int32_t* residual, int32_t* status, long long* work,
                                  int only_class, cudaStream_t stream) {
#define MOESCHED_GO(C)                                                                                         \
  do {                                                                                                         \
    if (work != nullptr)                                                                                       \
      return launch_warp_kernel(mw_kernel<C, MODE, true>, ge, B, stream, B, N, ge.S, demand, k_max, perm, dur, \
                                count, residual, status, work, only_class);                                    \
    return launch_warp_kernel(mw_kernel<C, MODE, false>, ge, B, stream, B, N, ge.S, demand, k_max, perm, dur,  \
                              count, residual, status, work, only_class);                                      \
  } while (0)
  switch (ge.cpl) {
    case 1: MOESCHED_GO(1);
    case 2: MOESCHED_GO(2);
    case 4: MOESCHED_GO(4);
    default: MOESCHED_GO(8);
  }
#undef MOESCHED_GO
}

// Batches with fewer matrices per SM than this go to the CTA-per-matrix kernel (N > 64). Measured on a
// B200: N = 256, B = 256 (1.7 per SM): 294 ms against 613 ms for one warp per matrix; N = 128, B = 1024
// (6.9 per SM): 91 ms against 63 ms -- with that many matrices per SM the warps of different matrices
// already fill the issue slots and the CTA's barriers only cost.
constexpr int MW_TEAM_MAX_PER_SM = 4;

cudaError_t run_mw(int B, int N, const int32_t* demand, int k_max, uint8_t* perm, int32_t* dur, int32_t* count,
                   int32_t* residual, int32_t* status, long long* work, cudaStream_t stream) {
  const Geometry ge = plan_geometry(N);
  int only_class = 0;
  if (N >= 48) {
    // Shared memory limits how many matrices an SM holds: first the matrices that fit 16-bit entries
    // (one CTA each at any N), then the rest as int32 (a 2-CTA cluster above N = 232).
    cudaError_t e = classify_matrices(B, N, demand, status, stream);
    if (e != cudaSuccess) return e;
    if (N > 64 && B < MW_TEAM_MAX_PER_SM * sm_count()) {
      // few large matrices: one CTA per matrix instead of one warp
      e = run_mw_team(B, N, demand, k_max, perm, dur, count, residual, status, work, stream);
    } else {
      Geometry g16 = ge;
      g16.cluster = false;
      g16.wpb = 1;
      g16.smem = warp_smem_bytes16(N, g16.S, g16.cpl);
      e = launch_mw_mode<2>(g16, B, N, demand, k_max, perm, dur, count, residual, status, work, CLASS_U16, stream);
    }
    if (e != cudaSuccess) return e;
    only_class = CLASS_I32;
  }
  if (ge.cluster) return launch_mw_mode<1>(ge, B, N, demand, k_max, perm, dur, count, residual, status, work,
                                           only_class, stream);
  return launch_mw_mode<0>(ge, B, N, demand, k_max, perm, dur, count, residual, status, work, only_class, stream);
}

}  // namespace moesched
