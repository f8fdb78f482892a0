// Birkhoff-von Neumann decomposition (paper Sec. 3.1) with one CTA of NW warps per demand matrix,
// for batches that have too few matrices to occupy the SMs with one warp each.
//
// Same method and same results as bvn_kernel.cu: north-west-corner padding, then per step the rows
// whose matched entry vanished are re-matched by the augmenting path whose lowest row is highest,
// the lexicographically smallest perfect matching is restored over the window of rows that
// changed, and the smallest matched entry is subtracted. Thread t owns row t and column t
// (team.cuh); the working copy of the matrix sits in the caller's global scratch slab.
#include "team.cuh"

namespace moesched {

namespace {

template <int NW>
struct BvnTeamShared {
  static constexpr int NT = 32 * NW;
  TeamShared<NW> team;
  unsigned char wait[NT];   // augmenting search: row met while below the threshold
  long long sums[2 * NT];   // row sums, then column sums
  int fill_cell[2 * NT];    // padded cells (offset into the working copy) and their amounts
  int fill_val[2 * NT];
};

}  // namespace

template <int NW>
__global__ void __launch_bounds__(32 * NW) bvn_team_kernel(int B, int N, int S, const int32_t* __restrict__ demand,
                                                           int k_max, uint8_t* __restrict__ perm,
                                                           int32_t* __restrict__ coef, int32_t* __restrict__ count,
                                                           int32_t* __restrict__ aug, int32_t* scratch,
                                                           int32_t* __restrict__ status,
                                                           long long* __restrict__ work_out) {
  constexpr int W = NW;
  constexpr int NT = 32 * NW;
  __shared__ BvnTeamShared<NW> bs;
  TeamShared<NW>& sh = bs.team;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int b = blockIdx.x;
  const bool in = t < N;
  TeamRed red;
  red.init(sh.red);

  unsigned work[MOESCHED_WORK_FIELDS];
#pragma unroll
  for (int q = 0; q < MOESCHED_WORK_FIELDS; ++q) work[q] = 0u;

  int* mat = scratch + (size_t)b * N * S;
  const int32_t* src = demand + (size_t)b * N * N;

  // ---- working copy, column sums (thread t: column t), row sums (one warp per row), validation ----
  long long cs = 0;
  int neg = 0;
  for (int r = 0; r < N; ++r) {
    if (t < S) {
      const int v = in ? src[(size_t)r * N + t] : 0;
      mat[(size_t)r * S + t] = v;
      cs += v;
      neg |= v < 0;
    }
  }
  for (int r = warp; r < N; r += NW) {
    long long part = 0;
    for (int c = lane; c < N; c += 32) part += src[(size_t)r * N + c];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(FULL, part, o);
    if (lane == 0) bs.sums[r] = part;
  }
  bs.sums[NT + t] = cs;
  sh.x[t] = -1;
  sh.mr[t] = -1;
  sh.lvl[t] = -1;
  red.open();
  __syncthreads();
  {
    // largest sum, clamped to 2^31 (anything above 2^31-1 is out of range)
    long long m = in ? max(bs.sums[t], cs) : 0;
    if (m < 0) m = 0;
    red.max_val(true, m > 2147483647LL ? 0x80000000u : (unsigned)m, lane);
    if (__any_sync(FULL, neg) && lane == 0) atomicOr(&red.cur()[TeamRed::SET], 1u);
  }
  red.close();
  const unsigned Tu = red.cur()[TeamRed::MAX];
  const bool any_neg = red.cur()[TeamRed::SET] != 0u;
  red.next();

  int st_code = MOESCHED_ST_OK;
  if (any_neg || Tu > 2147483647u) st_code = MOESCHED_ST_BAD_INPUT;
  int k = 0;

  if (st_code == MOESCHED_ST_OK) {
    const long long T = (long long)Tu;
    // ---- north-west-corner fill of the deficits: the staircase (at most 2N-1 cells) is walked by
    // one thread over the sums in shared memory, then all threads add the amounts in parallel ----
    if (t == 0) {
      int i = 0, j = 0, n = 0;
      long long a = T - bs.sums[0], bb = T - bs.sums[NT];
      for (int it = 0; it < 4 * N + 4 && i < N && j < N; ++it) {
        if (a == 0) { ++i; if (i < N) a = T - bs.sums[i]; continue; }
        if (bb == 0) { ++j; if (j < N) bb = T - bs.sums[NT + j]; continue; }
        const long long e = min(a, bb);
        if (n < 2 * NT) { bs.fill_cell[n] = i * S + j; bs.fill_val[n] = (int)e; ++n; }
        a -= e;
        bb -= e;
      }
      sh.misc[0] = n;
    }
    __syncthreads();
    {
      const int n = sh.misc[0];
      for (int q = t; q < n; q += NT) mat[bs.fill_cell[q]] += bs.fill_val[q];
    }
    __syncthreads();
    if (aug != nullptr && in) {
      int32_t* ao = aug + (size_t)b * N * N;
      for (int r = 0; r < N; ++r) ao[(size_t)r * N + t] = mat[(size_t)r * S + t];
    }

    // ---- support graph: Cc = rows with a positive entry in column t, Rr = columns of row t ----
    TeamMatch<NW> m;
#pragma unroll
    for (int w = 0; w < W; ++w) m.Cc[w] = m.Rr[w] = 0u;
    m.my_x = m.my_mr = -1;
    int mynz = 0;
    if (in) {
#pragma unroll
      for (int w = 0; w < W; ++w) {
        for (int q = 0; q < 32; ++q) {
          const int r = w * 32 + q;
          if (r >= N) break;
          if (mat[(size_t)r * S + t] > 0) { m.Cc[w] |= 1u << q; ++mynz; }
          if (mat[(size_t)t * S + r] > 0) m.Rr[w] |= 1u << q;
        }
      }
    }
    red.open();
    red.add_val((unsigned)mynz, lane);
    red.close();
    int nnz = (int)red.cur()[TeamRed::ADD];
    red.next();

    TeamMemo<NW> memo;
    memo.reset();
    int stamp = 0;   // base of the level stamps of the current backward search
    uint8_t* pout = perm + (size_t)b * k_max * N;
    int32_t* cout_ = coef + (size_t)b * k_max;
    int lo_changed = 0, hi_changed = N - 1;
    unsigned freerows[W];   // uniform: rows without a column
#pragma unroll
    for (int w = 0; w < W; ++w) {
      const int lo = w * 32;
      freerows[w] = N >= lo + 32 ? 0xffffffffu : (N <= lo ? 0u : (0xffffffffu >> (lo + 32 - N)));
    }

    while (nnz > 0 && k < k_max && st_code == MOESCHED_ST_OK) {
      // ---- re-match the free rows, lowest first ----
      if (t == 0) { sh.misc[2] = lo_changed; sh.misc[3] = hi_changed; }
      for (int outer = 0; outer < N; ++outer) {
        const int f = lowest_bit<W>(freerows);
        if (f < 0) break;
        // Augmenting search from row f over alternating paths of the support graph; among all
        // augmenting paths one whose lowest row is as high as possible: only rows >= thr are
        // expanded, and thr drops to the highest waiting row only when the search is stuck.
        int thr = f;
        bool visited = false;
        int jf = -1;
        bool stuck = false;
        bs.wait[t] = 0;
        unsigned xr[W];   // rows of the current frontier
#pragma unroll
        for (int w = 0; w < W; ++w) xr[w] = onehot_word(f, w);
        __syncthreads();
        for (int it = 0; it < 2 * N + 2; ++it) {
          red.open();
          bool isfree = false, met = false;
          if (in && !visited && meets<W>(m.Cc, xr)) {
            visited = true;
            unsigned hit[W];
#pragma unroll
            for (int w = 0; w < W; ++w) hit[w] = m.Cc[w] & xr[w];
            sh.par[t] = (short)lowest_bit<W>(hit);
            if (m.my_mr < 0) isfree = true;
            else if (m.my_mr >= thr) met = true;
            else bs.wait[MS_AT(m.my_mr, N)] = 1;
          }
          red.min_key(isfree, t, 0, lane);
          red.add_member<W>(met, m.my_mr, lane);
          red.close();
          const unsigned fkey = red.cur()[TeamRed::MIN];
          red.read_set<W>(xr);
          red.next();
          if (t == 0) work[WK_SCAN]++;
          if (fkey != 0xffffffffu) { jf = (int)(fkey >> 16); break; }
          if (!any_bit<W>(xr)) {
            // stuck: admit the highest waiting row, and only that one
            red.open();
            red.max_val(in && bs.wait[t] != 0, (unsigned)t + 1u, lane);
            red.close();
            const unsigned mx = red.cur()[TeamRed::MAX];
            red.next();
            if (mx == 0u) { stuck = true; break; }
            thr = (int)mx - 1;
            if (t == thr) bs.wait[t] = 0;
#pragma unroll
            for (int w = 0; w < W; ++w) xr[w] = onehot_word(thr, w);
          }
        }
        if (jf < 0 || stuck) { st_code = MOESCHED_ST_INTERNAL; break; }
        // flip the path back to row f: one thread walks it in shared memory
        if (t == 0) {
          int j = jf, ok = 0, lo = sh.misc[2], hi = sh.misc[3];
          for (int it = 0; it <= N; ++it) {
            const int i = MS_AT((int)sh.par[MS_AT(j, N)], N);
            const int jprev = sh.x[i];
            sh.mr[j] = (short)i;
            sh.x[i] = (short)j;
            lo = min(lo, i);
            hi = max(hi, i);
            work[WK_AUG]++;
            if (i == f) { ok = 1; break; }
            j = jprev;
            if (j < 0) break;
          }
          sh.misc[1] = ok;
          sh.misc[2] = lo;
          sh.misc[3] = hi;
        }
        __syncthreads();
        m.my_mr = sh.mr[t];
        {
          const int nx = sh.x[t];
          if (nx != m.my_x) memo.changed = true;
          m.my_x = nx;
        }
        if (!sh.misc[1]) { st_code = MOESCHED_ST_INTERNAL; break; }
        clear_bit<W>(freerows, f);
      }
      if (st_code != MOESCHED_ST_OK) break;
      if (any_bit<W>(freerows)) { st_code = MOESCHED_ST_INTERNAL; break; }
      __syncthreads();
      lo_changed = sh.misc[2];
      hi_changed = sh.misc[3];
      if (t == 0) work[WK_SKIP] += lo_changed;

      // ---- lexicographically smallest perfect matching over the window of changed rows ----
      if (!team_canonicalise<NW, true>(sh, red, N, t, lane, warp, in, m, memo, stamp, lo_changed, hi_changed,
                                       work)) {
        st_code = MOESCHED_ST_INTERNAL;
        break;
      }

      // ---- coefficient = smallest matched entry; subtract it along the matching; emit ----
      red.open();
      int val = INF32;
      if (in) val = mat[(size_t)MS_AT(m.my_mr, N) * S + t];
      {
        const unsigned wmin = __reduce_min_sync(FULL, (unsigned)val);
        if (lane == 0) atomicMin(&red.cur()[TeamRed::MIN], wmin);
      }
      red.close();
      const int cmin = (int)red.cur()[TeamRed::MIN];
      red.next();
      red.open();
      bool zero = false;
      if (in) {
        const int nv = val - cmin;
        mat[(size_t)MS_AT(m.my_mr, N) * S + t] = nv;
        zero = nv == 0;
        if (zero) {
#pragma unroll
          for (int w = 0; w < W; ++w) m.Cc[w] &= ~onehot_word(m.my_mr, w);
        }
        pout[(size_t)k * N + t] = (uint8_t)m.my_x;
      }
      if (t == 0) { cout_[k] = cmin; work[WK_MATCH]++; }
      ++k;
      red.add_member<W>(zero, m.my_mr, lane);
      red.add_val(zero ? 1u : 0u, lane);
      red.close();
      red.read_set<W>(freerows);
      nnz -= (int)red.cur()[TeamRed::ADD];
      red.next();
      // unmatch the rows whose entry vanished (thread c as the column, thread r as the row)
      if (zero) { m.my_mr = -1; sh.mr[t] = -1; }
      if (in && test_bit<W>(freerows, t)) {
#pragma unroll
        for (int w = 0; w < W; ++w) m.Rr[w] &= ~onehot_word(m.my_x, w);
        m.my_x = -1;
        sh.x[t] = -1;
      }
      lo_changed = N;
      hi_changed = -1;
      __syncthreads();
    }
    if (st_code == MOESCHED_ST_OK && nnz > 0) st_code = MOESCHED_ST_TRUNCATED;
  }

  if (st_code == MOESCHED_ST_BAD_INPUT) k = 0;
  if (t == 0) {
    count[b] = k;
    status[b] = st_code;
    if (work_out != nullptr) {
#pragma unroll
      for (int q = 0; q < MOESCHED_WORK_FIELDS; ++q) work_out[(size_t)b * MOESCHED_WORK_FIELDS + q] = work[q];
    }
  }
}

// ---- host side ---------------------------------------------------------------------------

template <int NW>
static cudaError_t launch_bvn_team(int B, int N, const int32_t* demand, int k_max, uint8_t* perm, int32_t* coef,
                                   int32_t* count, int32_t* aug, int32_t* scratch, int32_t* status, long long* work,
                                   cudaStream_t stream) {
  bvn_team_kernel<NW><<<B, 32 * NW, 0, stream>>>(B, N, bvn_scratch_stride(N), demand, k_max, perm, coef, count, aug,
                                                 scratch, status, work);
  return cudaGetLastError();
}

cudaError_t run_bvn_team(int B, int N, const int32_t* demand, int k_max, uint8_t* perm, int32_t* coef,
                         int32_t* count, int32_t* aug, int32_t* scratch, int32_t* status, long long* work,
                         cudaStream_t stream) {
  if (N <= 128) return launch_bvn_team<4>(B, N, demand, k_max, perm, coef, count, aug, scratch, status, work, stream);
  return launch_bvn_team<8>(B, N, demand, k_max, perm, coef, count, aug, scratch, status, work, stream);
}

}  // namespace moesched
