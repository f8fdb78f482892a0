// Greedy max-weight decomposition (paper Sec. 3.2) with one CTA of NW warps per demand matrix, for
// matrices above 64 ranks whose entries fit 16 bits: the residual matrix sits in shared memory as
// 16-bit entries, thread t owns column t (its dual, its distance in the current search) and row t.
//
// Same method and same results as mw_kernel.cu. Per greedy step:
//   1. the column duals carry over from the previous step (weights only decreased, so they are still
//      feasible) and are shifted so that the largest is zero;
//   2. every row bids for the column with its smallest reduced cost; a column takes the lowest bidder;
//      rows left over then bid, round after round, for the lowest column that is tight for them and
//      still free (a maximal matching of the tight graph, all rows at once);
//   3. every row still left over is inserted by a shortest-augmenting-path search (Jonker-Volgenant style,
//      column duals only) that settles ALL columns at the current minimum distance at once: they are
//      found with one barrier (per-warp minimum and ballot, then every thread combines the warps'
//      entries), and every thread then relaxes its own column against the rows of the settled
//      columns one after the other without further barriers. On sparse matrices with many equal
//      entries most settled columns come in such groups;
//   4. row duals = row minima of the reduced costs, tight edges = entries that attain them; the
//      lexicographically smallest perfect matching of that graph (team_canonicalise_par) is the step's
//      matching, whatever optimal duals and matching the solver arrived at;
//   5. the matched entries are served whole, the largest one is the matching's duration.
#include "team.cuh"

namespace moesched {

namespace {

template <int NW>
struct MwTeamShared {
  static constexpr int NT = 32 * NW;
  TeamShared<NW> team;
  TeamSearchShared<NW> search;   // tight graph as bit matrices, per-warp search marks
  int vs[NT];               // column duals, published for the row-wise passes
  int u[NT];                // row duals: smallest reduced cost of the row
  int first[NT];            // lowest row that bid for the column
  int hbuf[2][NT];          // reduced cost of the column's own matched entry (two buffers, see the search)
  int wmin[2][NW];          // per warp: smallest distance among its unsettled columns
  unsigned wcand[2][NW];    // per warp: the lanes that attain it
  short best[NT];           // column each row bids for
};

// The duals stay within [-2^30, 0] (see solve_assignment in mw_kernel.cu); shifted by this they are
// positive and can go through the unsigned maximum of the reduction slots.
constexpr int DUAL_BIAS = 0x60000000;

// Smallest reduced cost of one row and the lowest column attaining it; every lane returns both.
template <int NW>
__device__ __forceinline__ void row_minimum(const unsigned short* Rrow, const int* vs, int N, int lane, int& mn,
                                            int& col) {
  int lmin = INF32, lcol = INF32;
#pragma unroll
  for (int q = 0; q < NW; ++q) {
    const int c = q * 32 + lane;
    if (c < N) {
      const int d = -(int)Rrow[c] - vs[c];
      if (d < lmin) { lmin = d; lcol = c; }
    }
  }
  mn = __reduce_min_sync(FULL, lmin);
  col = __reduce_min_sync(FULL, lmin == mn ? lcol : INF32);
}

// Tight edges under the column duals (thread t: v of column t) and the row duals ms.u: entry (r, t) is
// tight iff its reduced cost equals the row's smallest. Leaves the graph as bit matrices in shared
// memory (by columns and by rows) and in m.Cc / m.Rr. Ends with a barrier.
template <int NW>
__device__ __forceinline__ void tight_graph_team(const unsigned short* R, MwTeamShared<NW>& ms, int N, int t, int lane,
                                                 int warp, bool in, int v, TeamMatch<NW>& m) {
  constexpr int W = NW;
#pragma unroll
  for (int w = 0; w < W; ++w) {
    unsigned cc = 0u;
    for (int q = 0; q < 32; ++q) {
      const int r = w * 32 + q;
      if (r >= N) break;
      const bool tight = in && (-(int)R[(size_t)r * N + t] - v == ms.u[r]);
      const unsigned rowword = __ballot_sync(FULL, tight);
      if (lane == 0) ms.search.rr[r * NW + warp] = rowword;
      cc |= tight ? 1u << q : 0u;
    }
    m.Cc[w] = cc;
    ms.search.cc[t * NW + w] = cc;
  }
  __syncthreads();
#pragma unroll
  for (int w = 0; w < W; ++w) m.Rr[w] = in ? ms.search.rr[t * NW + w] : 0u;
}

}  // namespace

template <int NW, bool COUNT>
__global__ void __launch_bounds__(32 * NW) mw_team_kernel(int B, int N, const int32_t* __restrict__ demand, int k_max,
                                                          uint8_t* __restrict__ perm, int32_t* __restrict__ dur,
                                                          int32_t* __restrict__ count, int32_t* __restrict__ residual,
                                                          int32_t* status, long long* __restrict__ work_out) {
  constexpr int W = NW;
  constexpr int NT = 32 * NW;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ MwTeamShared<NW> ms;
  TeamShared<NW>& sh = ms.team;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int b = blockIdx.x;
  if (status[b] != CLASS_U16) return;   // uniform: wide matrices are left to the one-warp kernels
  unsigned short* R = reinterpret_cast<unsigned short*>(smem_raw);
  const bool in = t < N;
  TeamRed red;
  red.init(sh.red);

  unsigned work[MOESCHED_WORK_FIELDS];
#pragma unroll
  for (int q = 0; q < MOESCHED_WORK_FIELDS; ++q) work[q] = 0u;

  // ---- residual matrix into shared memory (the class pre-pass guarantees 0 <= entry <= 65535) ----
  const int32_t* src = demand + (size_t)b * N * N;
  int mynz = 0;
  for (int e = t; e < N * N; e += NT) {
    const int val = src[e];
    R[e] = (unsigned short)val;
    mynz += val != 0;
  }
  sh.x[t] = -1;
  sh.mr[t] = -1;
  sh.lvl[t] = -1;
#pragma unroll
  for (int w = 0; w < W; ++w) ms.search.lvl[w][t] = -1;
  red.open();
  red.add_val((unsigned)mynz, lane);
  red.close();
  int nnz = (int)red.cur()[TeamRed::ADD];
  red.next();

  int st_code = MOESCHED_ST_OK;
  int k = 0;
  int v = 0;        // dual of column t (cost problem: cost = -R)
  int stamp = 0;    // base of the level stamps of the canonicalisation searches
  uint8_t* pout = perm + (size_t)b * k_max * N;
  int32_t* dout = dur + (size_t)b * k_max;
  TeamMatch<NW> m;

  while (k < k_max && nnz > 0 && st_code == MOESCHED_ST_OK) {
    // ---- 1. shift the duals so that the largest is zero; publish them ----
    red.open();
    red.max_val(in, (unsigned)(v + DUAL_BIAS), lane);
    ms.first[t] = INF32;
    red.close();
    v -= (int)red.cur()[TeamRed::MAX] - DUAL_BIAS;
    red.next();
    ms.vs[t] = in ? v : 0;
    __syncthreads();

    // ---- 2. bids: every row names its best column, a column takes the lowest row that named it ----
    for (int r = warp; r < N; r += NW) {
      int mn, col;
      row_minimum<NW>(R + (size_t)r * N, ms.vs, N, lane, mn, col);
      if (lane == 0) { ms.best[r] = (short)col; ms.u[r] = mn; }
    }
    __syncthreads();
    if (in) atomicMin(&ms.first[MS_AT((int)ms.best[t], N)], t);
    __syncthreads();
    int my_mr = in && ms.first[t] != INF32 ? ms.first[t] : -1;   // row of column t
    int my_x = in && ms.first[MS_AT((int)ms.best[t], N)] == t ? (int)ms.best[t] : -1;   // column of row t
    if (t == 0) work[WK_TIGHT] += N;
    // tight edges under the current duals, by rows: the leftover rows bid for free tight columns
    tight_graph_team<NW>(R, ms, N, t, lane, warp, in, v, m);
    unsigned freecols[W], freerows[W];
    for (int round = 0; round < N; ++round) {
      red.open();
      red.add_member<W>(in && my_mr < 0, t, lane);
      ms.first[t] = INF32;
      red.close();
      red.read_set<W>(freecols);
      red.next();
      int bid = -1;
      if (in && my_x < 0) {
        unsigned open_[W];
#pragma unroll
        for (int w = 0; w < W; ++w) open_[w] = m.Rr[w] & freecols[w];
        bid = lowest_bit<W>(open_);
      }
      red.open();
      if (bid >= 0) atomicMin(&ms.first[bid], t);
      red.add_val(bid >= 0 ? 1u : 0u, lane);
      red.close();
      const unsigned bids = red.cur()[TeamRed::ADD];
      red.next();
      if (bids == 0u) break;
      if (in && my_mr < 0 && ms.first[t] != INF32) my_mr = ms.first[t];
      if (bid >= 0 && ms.first[bid] == t) my_x = bid;
      __syncthreads();   // first[] is cleared at the top of the next round
    }
    sh.mr[t] = (short)my_mr;
    sh.x[t] = (short)my_x;
    red.open();
    red.add_member<W>(in && my_x < 0, t, lane);
    red.close();
    red.read_set<W>(freerows);
    red.next();

    // ---- 3. the rows still left over, lowest first: shortest augmenting path, settling whole groups ----
    for (int outer = 0; outer < N && st_code == MOESCHED_ST_OK; ++outer) {
      const int f = lowest_bit<W>(freerows);
      if (f < 0) break;
      clear_bit<W>(freerows, f);
      int dist = in ? -(int)R[(size_t)f * N + t] - v : INF32;
      int pred = f;
      bool done = !in;
      int jfin = -1, mu = 0;
      for (int it = 0; it <= N && jfin < 0; ++it) {
        const int p = it & 1;
        // candidates of this warp: the unsettled columns at the warp's smallest distance; each
        // publishes the reduced cost of its own matched entry, which the relaxation below needs
        const int d_eff = done ? INF32 : dist;
        const int wm = __reduce_min_sync(FULL, d_eff);
        const bool cand = !done && dist == wm;
        const unsigned cb = __ballot_sync(FULL, cand);
        if (cand) ms.hbuf[p][t] = my_mr >= 0 ? -(int)R[(size_t)MS_AT(my_mr, N) * N + t] - v : 0;
        if (lane == 0) { ms.wmin[p][warp] = wm; ms.wcand[p][warp] = cb; }
        __syncthreads();
        mu = INF32;
#pragma unroll
        for (int w = 0; w < W; ++w) mu = min(mu, ms.wmin[p][w]);
        if (mu == INF32) break;   // nothing left to settle and no free column met: cannot happen
        if (t == 0) work[WK_BATCH]++;
        // every column at distance mu is settled now
        unsigned S[W], hit[W];
#pragma unroll
        for (int w = 0; w < W; ++w) {
          S[w] = ms.wmin[p][w] == mu ? ms.wcand[p][w] : 0u;
          hit[w] = S[w] & freecols[w];
        }
        if ((S[warp] >> lane) & 1u) done = true;   // (S[warp]: the compiler selects the word, W is small)
        jfin = lowest_bit<W>(hit);
        if (jfin >= 0) break;   // a free column at the smallest distance: path found
        // all of them are matched: relax against their rows, four at a time so that the loads overlap
#pragma unroll
        for (int w = 0; w < W; ++w) {
          unsigned sw = S[w];
          while (sw != 0u) {
            int cq[4], iq[4], hq[4], vq[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              cq[q] = sw != 0u ? w * 32 + __ffs(sw) - 1 : -1;
              sw &= sw - 1u;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              iq[q] = cq[q] >= 0 ? MS_AT((int)sh.mr[cq[q]], N) : 0;
              hq[q] = cq[q] >= 0 ? ms.hbuf[p][cq[q]] - mu : 0;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) vq[q] = R[(size_t)iq[q] * N + (in ? t : 0)];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int nd = -vq[q] - v - hq[q];
              if (cq[q] >= 0 && !done && nd < dist) { dist = nd; pred = iq[q]; }
            }
            if (t == 0) work[WK_SCAN] += (cq[0] >= 0) + (cq[1] >= 0) + (cq[2] >= 0) + (cq[3] >= 0);
          }
        }
      }
      if (jfin < 0) { st_code = MOESCHED_ST_INTERNAL; break; }
      clear_bit<W>(freecols, jfin);
      // settled columns move their dual so that the shortest-path tree stays tight
      if (done && in) v += dist - mu;
      sh.par[t] = (short)pred;
      __syncthreads();
      // flip the path back to row f: one thread walks it in shared memory
      if (t == 0) {
        int j = jfin, ok = 0;
        for (int it = 0; it <= N; ++it) {
          const int i = MS_AT((int)sh.par[MS_AT(j, N)], N);
          const int jprev = sh.x[i];
          sh.mr[j] = (short)i;
          sh.x[i] = (short)j;
          if (i == f) { ok = 1; break; }
          j = jprev;
          if (j < 0) break;
        }
        sh.misc[1] = ok;
        work[WK_AUG]++;
      }
      __syncthreads();
      my_mr = sh.mr[t];
      if (!sh.misc[1]) st_code = MOESCHED_ST_INTERNAL;
    }
    if (st_code != MOESCHED_ST_OK) break;

    // ---- 4. row duals, tight edges, lexicographically smallest optimal matching ----
    ms.vs[t] = in ? v : 0;
    __syncthreads();
    for (int r = warp; r < N; r += NW) {
      int mn, col;
      row_minimum<NW>(R + (size_t)r * N, ms.vs, N, lane, mn, col);
      if (lane == 0) ms.u[r] = mn;
    }
    __syncthreads();
    tight_graph_team<NW>(R, ms, N, t, lane, warp, in, v, m);
    m.my_x = sh.x[t];
    m.my_mr = sh.mr[t];
    if (!team_canonicalise_par<NW>(sh, ms.search, red, N, t, lane, warp, in, m, stamp, 0, work)) {
      st_code = MOESCHED_ST_INTERNAL;
      break;
    }

    // ---- 5. serve: the heaviest matched pair sets the duration; matched entries are sent whole ----
    red.open();
    int val = 0;
    if (in && m.my_mr >= 0) {
      val = R[(size_t)MS_AT(m.my_mr, N) * N + t];
      R[(size_t)MS_AT(m.my_mr, N) * N + t] = 0;
      pout[(size_t)k * N + t] = (uint8_t)m.my_x;
    }
    red.max_val(val > 0, (unsigned)val, lane);
    red.add_val(val != 0 ? 1u : 0u, lane);
    red.close();
    if (t == 0) { dout[k] = (int)red.cur()[TeamRed::MAX]; work[WK_MATCH]++; }
    nnz -= (int)red.cur()[TeamRed::ADD];
    red.next();
    ++k;
  }
  if (st_code == MOESCHED_ST_OK && nnz > 0) st_code = MOESCHED_ST_TRUNCATED;

  __syncthreads();
  if (t == 0) {
    count[b] = k;
    status[b] = st_code;
    if constexpr (COUNT) {
      if (work_out != nullptr) {
#pragma unroll
        for (int q = 0; q < MOESCHED_WORK_FIELDS; ++q) work_out[(size_t)b * MOESCHED_WORK_FIELDS + q] = work[q];
      }
    }
  }
  if (residual != nullptr) {
    int32_t* ro = residual + (size_t)b * N * N;
    for (int e = t; e < N * N; e += NT) ro[e] = R[e];
  }
}

// ---- host side ---------------------------------------------------------------------------

template <int NW>
static cudaError_t launch_mw_team(int B, int N, const int32_t* demand, int k_max, uint8_t* perm, int32_t* dur,
                                  int32_t* count, int32_t* residual, int32_t* status, long long* work,
                                  cudaStream_t stream) {
  const size_t smem = align16((size_t)N * N * 2);
  cudaError_t e;
  if (work != nullptr) {
    e = cudaFuncSetAttribute(mw_team_kernel<NW, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    mw_team_kernel<NW, true><<<B, 32 * NW, smem, stream>>>(B, N, demand, k_max, perm, dur, count, residual, status,
                                                           work);
  } else {
    e = cudaFuncSetAttribute(mw_team_kernel<NW, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    mw_team_kernel<NW, false><<<B, 32 * NW, smem, stream>>>(B, N, demand, k_max, perm, dur, count, residual, status,
                                                            work);
  }
  return cudaGetLastError();
}

// Decomposes the matrices whose status holds CLASS_U16 (64 < N <= 256); the others are left untouched.
cudaError_t run_mw_team(int B, int N, const int32_t* demand, int k_max, uint8_t* perm, int32_t* dur, int32_t* count,
                        int32_t* residual, int32_t* status, long long* work, cudaStream_t stream) {
  if (N <= 128) return launch_mw_team<4>(B, N, demand, k_max, perm, dur, count, residual, status, work, stream);
  return launch_mw_team<8>(B, N, demand, k_max, perm, dur, count, residual, status, work, stream);
}

}  // namespace moesched
