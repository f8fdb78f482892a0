// Building blocks for the kernels in which a TEAM of NW warps (one CTA) owns one demand matrix.
// They serve batches with too few matrices to fill the SMs with one warp per matrix (N > 128 in
// the benchmarked configurations). Thread t of the CTA owns row t and column t of the matrix: its
// adjacency to the columns (Rr) and to the rows (Cc) as bit masks of W = NW words in registers, its
// matched column and row as scalars. Sets of rows or columns that all threads need are built in
// shared memory with one atomic per member and read back after a CTA barrier; membership that
// only the owner needs stays a flag in the owner's registers. Every value a branch depends on is
// read from shared memory after a barrier, so control flow is uniform across the CTA and every
// barrier is reached by all of its threads.
#pragma once

#include "common.cuh"

namespace moesched {

// Reduction slots in shared memory, three deep so that one barrier per phase is enough: in phase p
// the threads clear the slot of phase p+1 (last read before the barrier of phase p-1), add to the
// slot of phase p, meet at the barrier and read the slot of phase p.
struct TeamRed {
  static constexpr int SET = 0;    // words 0..7: a set of rows or columns (bitwise OR)
  static constexpr int MIN = 8;    // unsigned minimum (starts at 0xffffffff)
  static constexpr int ADD = 9;    // sum
  static constexpr int MAX = 10;   // unsigned maximum
  static constexpr int SLOT = 12;
  unsigned* buf;   // 3 * SLOT words
  int which;       // slot of the current phase: 0, 1, 2 (uniform)

  __device__ __forceinline__ void init(unsigned* shared_words) {
    buf = shared_words;
    which = 0;
    if (threadIdx.x < 3 * SLOT) buf[threadIdx.x] = (threadIdx.x % SLOT) == MIN ? 0xffffffffu : 0u;
    __syncthreads();
  }
  __device__ __forceinline__ unsigned* cur() const { return buf + which * SLOT; }
  // start of a phase: clear the slot the next phase will use
  __device__ __forceinline__ void open() const {
    const int nx = which == 2 ? 0 : which + 1;
    if (threadIdx.x < SLOT) buf[nx * SLOT + threadIdx.x] = threadIdx.x == MIN ? 0xffffffffu : 0u;
  }
  // all contributions made: after this the slot may be read
  __device__ __forceinline__ void close() const { __syncthreads(); }
  // the slot has been read
  __device__ __forceinline__ void next() { which = which == 2 ? 0 : which + 1; }

  // member `index` joins the set if flag; a warp with many joiners combines them first
  template <int W>
  __device__ __forceinline__ void add_member(bool flag, int index, int lane) const {
    const unsigned ball = __ballot_sync(FULL, flag);
    if (ball == 0u) return;
    unsigned* s = cur() + SET;
    if (__popc(ball) <= 4) {
      if (flag) atomicOr(&s[index >> 5], 1u << (index & 31));
    } else {
      unsigned mine = 0u;
#pragma unroll
      for (int w = 0; w < W; ++w) {
        const unsigned r = __reduce_or_sync(FULL, flag ? onehot_word(index, w) : 0u);
        if (lane == w) mine = r;
      }
      if (lane < W && mine != 0u) atomicOr(&s[lane], mine);
    }
  }
  template <int W>
  __device__ __forceinline__ void read_set(unsigned (&out)[W]) const {
#pragma unroll
    for (int w = 0; w < W; ++w) out[w] = cur()[SET + w];
  }
  // lowest index among the flagged threads, packed with a 16-bit payload: index << 16 | payload
  __device__ __forceinline__ void min_key(bool flag, int index, int payload, int lane) const {
    const unsigned ball = __ballot_sync(FULL, flag);
    if (ball == 0u) return;
    if (lane == __ffs(ball) - 1) atomicMin(&cur()[MIN], ((unsigned)index << 16) | ((unsigned)payload & 0xffffu));
  }
  __device__ __forceinline__ void max_val(bool flag, unsigned v, int lane) const {
    const unsigned m = __reduce_max_sync(FULL, flag ? v : 0u);
    if (lane == 0 && m != 0u) atomicMax(&cur()[MAX], m);
  }
  __device__ __forceinline__ void add_val(unsigned v, int lane) const {
    const unsigned m = __reduce_add_sync(FULL, v);
    if (lane == 0 && m != 0u) atomicAdd(&cur()[ADD], m);
  }
};

template <int NW>
struct TeamShared {
  static constexpr int NT = 32 * NW;
  short x[NT];            // row -> column (-1: none)
  short mr[NT];           // column -> row (-1: none)
  short par[NT];          // augmenting search: row from which a column was reached
  int lvl[NT];            // stamp of the backward-search level at which a row was reached
  unsigned red[3 * TeamRed::SLOT];
  unsigned tot[NW * NW];  // per-warp column sets of the candidate test
  unsigned ri[NW];        // columns adjacent to the row being searched
  int misc[8];
};

template <int W>
__device__ __forceinline__ bool meets(const unsigned (&a)[W], const unsigned (&b)[W]) {
  unsigned o = 0u;
#pragma unroll
  for (int w = 0; w < W; ++w) o |= a[w] & b[w];
  return o != 0u;
}

// The matching of one team: who is matched to whom, as the owner thread sees it.
template <int NW>
struct TeamMatch {
  static constexpr int W = NW;
  unsigned Rr[W];   // columns adjacent to row t
  unsigned Cc[W];   // rows adjacent to column t
  int my_x;         // column of row t (-1: free)
  int my_mr;        // row of column t (-1: free)
};

// Rows that could move to a lower column: row r qualifies iff it is adjacent to a column below its
// own whose row lies above r. The columns matched to rows above r are an exclusive suffix OR over
// the threads: inside the warp by shuffles, across warps through shared memory. One barrier.
template <int NW>
__device__ __forceinline__ bool team_is_candidate(TeamShared<NW>& sh, int t, int lane, int warp, bool in,
                                                  const TeamMatch<NW>& m) {
  constexpr int W = NW;
  unsigned v[W];
#pragma unroll
  for (int w = 0; w < W; ++w) v[w] = in ? onehot_word(m.my_x, w) : 0u;
#pragma unroll
  for (int w = 0; w < W; ++w) {
#pragma unroll
    // (a lane whose source would lie beyond lane 31 gets its own value back: harmless in an OR)
    for (int o = 1; o < 32; o <<= 1) v[w] |= __shfl_down_sync(FULL, v[w], o);
  }
  unsigned above[W];
#pragma unroll
  for (int w = 0; w < W; ++w) {
    // v covers this row and all higher rows of the warp; a column is matched to one row only, so
    // taking the row's own column out leaves exactly the columns of the higher rows
    above[w] = v[w] & ~(in ? onehot_word(m.my_x, w) : 0u);
    const unsigned total = __shfl_sync(FULL, v[w], 0);
    if (lane == w) sh.tot[warp * W + w] = total;
  }
  __syncthreads();
  for (int g = warp + 1; g < NW; ++g) {
#pragma unroll
    for (int w = 0; w < W; ++w) above[w] |= sh.tot[g * W + w];
  }
  if (!in || m.my_x < 0) return false;
  unsigned o = 0u;
#pragma unroll
  for (int w = 0; w < W; ++w) o |= m.Rr[w] & above[w] & ~ge_word(m.my_x, w);
  return o != 0u;
}

// Memo carried from one call of team_canonicalise to the next when the graph only loses edges
// between calls (Birkhoff), the counterpart of CanonMemo in common.cuh spread over the row owners:
// known = row t's last search found no lower column and none of the rows that could reach it has
// changed column since; dep = the searched rows whose recorded set contains row t; changed = row
// t's column changed since the last call.
template <int NW>
struct TeamMemo {
  bool known, changed;
  unsigned dep[NW];
  __device__ __forceinline__ void reset() {
    known = changed = false;
#pragma unroll
    for (int w = 0; w < NW; ++w) dep[w] = 0u;
  }
};

// One phase: the rows flagged `moved` void every record that contains them (and their own).
template <int NW>
__device__ __forceinline__ void team_void_records(TeamRed& red, int t, bool moved, TeamMemo<NW>& memo) {
  constexpr int W = NW;
  red.open();
  if (moved) {
    unsigned* s = red.cur() + TeamRed::SET;
#pragma unroll
    for (int w = 0; w < W; ++w) {
      const unsigned v = memo.dep[w] | onehot_word(t, w);
      if (v != 0u) atomicOr(&s[w], v);
      memo.dep[w] = 0u;
    }
  }
  red.close();
  if ((red.cur()[TeamRed::SET + (t >> 5)] >> (t & 31)) & 1u) memo.known = false;
  red.next();
}

// Lexicographically smallest perfect matching of the graph (Rr / Cc) over the window of rows
// [start, last], given a perfect matching that already equals the answer below `start` (see
// canonicalise() in common.cuh for the argument; this is the same procedure with the sets spread
// over the CTA). For each row i that could move: the rows >= i that reach i by alternating steps
// are found level by level -- a row joins when it is adjacent to the column of a row of the
// previous level -- then row i takes the lowest adjacent column whose row was reached and the
// matching is rotated along the cycle. Returns false if an iteration limit was hit. Uniform.
template <int NW, bool MEMO>
__device__ __forceinline__ bool team_canonicalise(TeamShared<NW>& sh, TeamRed& red, int N, int t, int lane, int warp,
                                                  bool in, TeamMatch<NW>& m, TeamMemo<NW>& memo, int& stamp,
                                                  int start, int last, unsigned (&work)[MOESCHED_WORK_FIELDS]) {
  constexpr int W = NW;
  bool ok_all = true;
  if constexpr (MEMO) {
    team_void_records<NW>(red, t, memo.changed, memo);
    memo.changed = false;
  }
  bool cand = team_is_candidate<NW>(sh, t, lane, warp, in, m);
  int from = start;
  for (int guard = 0; guard < N; ++guard) {
    // next row that could move
    red.open();
    red.min_key(cand && t >= from && t <= last && !(MEMO && memo.known), t, 0, lane);
    red.close();
    const unsigned ikey = red.cur()[TeamRed::MIN];
    red.next();
    if (ikey == 0xffffffffu) break;
    const int i = (int)(ikey >> 16);
    from = i + 1;
    if (t == 0) { work[WK_SWEEP]++; work[WK_POP]++; }
    // Every search takes a fresh range of N + 2 level stamps, so that the marks of earlier searches
    // never need clearing. Before the stamps could pass 2^31 (after some 8 million searches at
    // N = 256; a complete worst-case decomposition can get there) all marks are wiped and the
    // stamps start over. stamp is uniform, so every thread takes this branch or none does.
    if (stamp > 0x7f000000) {
      __syncthreads();
      sh.lvl[t] = -1;
      stamp = 0;
      __syncthreads();
    }
    stamp += N + 2;
    // level 0: row i itself. Its adjacency is published for the column choice (read several
    // barriers later; the previous search's readers are past the barrier above).
    bool in_anc = t == i;
    if (t == i) {
      sh.lvl[i] = stamp;
#pragma unroll
      for (int w = 0; w < W; ++w) sh.ri[w] = m.Rr[w];
    }
    const int xi = sh.x[i];
    unsigned xf[W];   // columns of the rows of the current level
#pragma unroll
    for (int w = 0; w < W; ++w) xf[w] = onehot_word(xi, w);
    int level = 0;
    for (int it = 0; it < N; ++it) {
      red.open();
      const bool isnew = in && t > i && !in_anc && meets<W>(m.Rr, xf);
      if (isnew) {
        in_anc = true;
        sh.lvl[t] = stamp + level + 1;
      }
      red.add_member<W>(isnew, m.my_x, lane);
      red.close();
      red.read_set<W>(xf);
      red.next();
      if (t == 0) {
        work[WK_LEVEL]++;
#pragma unroll
        for (int w = 0; w < W; ++w) work[WK_POP] += __popc(xf[w]);
      }
      if (!any_bit<W>(xf)) break;
      ++level;
    }
    // lowest column row i may take: adjacent to i, its row reached (its own column always qualifies)
    red.open();
    {
      const bool adj = in && ((sh.ri[t >> 5] >> (t & 31)) & 1u);
      const bool reached = adj && m.my_mr >= 0 && sh.lvl[MS_AT(m.my_mr, N)] >= stamp;
      red.min_key(reached, t, m.my_mr, lane);
    }
    red.close();
    const unsigned key = red.cur()[TeamRed::MIN];
    red.next();
    if (key == 0xffffffffu) { ok_all = false; continue; }
    const int jstar = MS_AT((int)(key >> 16), N);
    if (jstar == xi) {
      // record: row i stays put until one of the rows that can reach it changes column
      if constexpr (MEMO) {
        if (in_anc) {
#pragma unroll
          for (int w = 0; w < W; ++w) memo.dep[w] |= onehot_word(i, w);
        }
        if (t == i) memo.known = true;
      }
      continue;
    }
    // rotate along the alternating cycle: the row that gives up column jstar takes the column of
    // its successor towards row i, and so on down the levels
    int cur = MS_AT((int)(key & 0xffffu), N);
    int lvl = sh.lvl[cur] - stamp;
    if (lvl <= 0 || lvl > level) { ok_all = false; continue; }
    for (int it = 0; it < N && lvl > 0; ++it) {
      red.open();
      const bool q = in && m.my_mr >= 0 && sh.lvl[MS_AT(m.my_mr, N)] == stamp + lvl - 1 && test_bit<W>(m.Cc, cur);
      red.min_key(q, t, m.my_mr, lane);
      red.close();
      const unsigned k2 = red.cur()[TeamRed::MIN];
      red.next();
      if (k2 == 0xffffffffu) { ok_all = false; break; }
      const int c2 = MS_AT((int)(k2 >> 16), N), nxt = MS_AT((int)(k2 & 0xffffu), N);
      if (t == c2) {
        m.my_mr = cur;
        sh.mr[c2] = (short)cur;
        sh.x[cur] = (short)c2;
      }
      last = max(last, cur);
      cur = nxt;
      --lvl;
      if (t == 0) work[WK_ROT]++;
    }
    if (t == jstar) {
      m.my_mr = i;
      sh.mr[jstar] = (short)i;
      sh.x[i] = (short)jstar;
    }
    __syncthreads();
    {
      const int nx = sh.x[t];
      const bool moved = nx != m.my_x;
      m.my_x = nx;
      // the moved rows changed column: every record that contains one of them is void
      if constexpr (MEMO) team_void_records<NW>(red, t, moved, memo);
    }
    cand = team_is_candidate<NW>(sh, t, lane, warp, in, m);
  }
  return ok_all;
}


// ---- canonicalisation with one search per WARP, several rows searched at once -----------------------
//
// The graph is held as bit matrices in shared memory (cc: rows adjacent to each column, rr: columns
// adjacent to each row) next to x / mr. A backward search then needs no exchange between warps: the
// lanes of ONE warp each look after the rows w * 32 + lane, a frontier row contributes the row set of
// its matched column with two vector loads, and an OR-reduction per word gives the next level. The NW
// warps of the CTA search the NW lowest rows that could move at the same time, each as if it were the
// only one. That is exact as long as no searched row moves: a search for row i looks at the rows above
// i and the current matching only. The results are then taken in row order up to the first row that
// does move; that warp rotates the matching along its cycle, the searches of the rows behind it are
// thrown away and the rows that could move are determined anew.
template <int NW>
struct TeamSearchShared {
  static constexpr int NT = 32 * NW;
  unsigned cc[NT * NW];     // word w of the rows adjacent to column c at cc[c * NW + w]
  unsigned rr[NT * NW];     // word w of the columns adjacent to row r at rr[r * NW + w]
  int lvl[NW][NT];          // per warp: stamp of the level at which its search reached a row
  int res[NW][4];           // per warp: row searched, column found, levels, rows reached
};

// The k-th lowest member (k = 0 for the lowest) of a set, or -1 if it has no more than k members.
template <int W>
__device__ __forceinline__ int kth_member(const unsigned (&m)[W], int k) {
  int r = -1, seen = 0;
#pragma unroll
  for (int w = 0; w < W; ++w) {
    const int pc = __popc(m[w]);
    if (r < 0 && k < seen + pc) {
      unsigned v = m[w];
      for (int q = seen; q < k; ++q) v &= v - 1u;
      r = w * 32 + __ffs(v) - 1;
    }
    seen += pc;
  }
  return r;
}

template <int W>
__device__ __forceinline__ void load_words(const unsigned* p, unsigned (&out)[W]) {
  if constexpr (W % 4 == 0) {
#pragma unroll
    for (int q = 0; q < W / 4; ++q) {
      const uint4 v = reinterpret_cast<const uint4*>(p)[q];
      out[4 * q] = v.x; out[4 * q + 1] = v.y; out[4 * q + 2] = v.z; out[4 * q + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int w = 0; w < W; ++w) out[w] = p[w];
  }
}

// Backward search from row i among the rows above it (one warp; every lane returns the same values):
// the lowest column that row i can take in a perfect matching that keeps the rows below i where they
// are, or -1 if an iteration limit was hit. lvl[r] = stamp + level for every row reached (row i: stamp).
template <int NW>
__device__ __forceinline__ int warp_back_search(const TeamShared<NW>& sh, const TeamSearchShared<NW>& ts, int* lvl,
                                                int stamp, int N, int i, int lane, int& levels, int& reached) {
  constexpr int W = NW;
  unsigned anc[W], F[W];
#pragma unroll
  for (int w = 0; w < W; ++w) anc[w] = F[w] = onehot_word(i, w);
  if (lane == 0) lvl[i] = stamp;
  int level = 0;
  levels = 0;
  reached = 1;
  for (int it = 0; it < N; ++it) {
    unsigned acc[W];
#pragma unroll
    for (int w = 0; w < W; ++w) acc[w] = 0u;
#pragma unroll
    for (int w = 0; w < W; ++w) {
      if ((F[w] >> lane) & 1u) {
        const int c = MS_AT((int)sh.x[w * 32 + lane], N);
        unsigned col[W];
        load_words<W>(ts.cc + c * W, col);
#pragma unroll
        for (int q = 0; q < W; ++q) acc[q] |= col[q];
      }
    }
    bool grew = false;
#pragma unroll
    for (int w = 0; w < W; ++w) {
      const unsigned a = __reduce_or_sync(FULL, acc[w]) & ge_word(i + 1, w) & ~anc[w];
      anc[w] |= a;
      F[w] = a;
      grew |= a != 0u;
      reached += __popc(a);
    }
    ++levels;
    if (!grew) break;
    ++level;
#pragma unroll
    for (int w = 0; w < W; ++w)
      if ((F[w] >> lane) & 1u) lvl[MS_AT(w * 32 + lane, N)] = stamp + level;
  }
  __syncwarp();
  // lowest column adjacent to row i whose row was reached (its own column always qualifies)
  int jstar = -1;
#pragma unroll
  for (int w = 0; w < W; ++w) {
    const int c = w * 32 + lane;
    bool ok = false;
    if (c < N && ((ts.rr[i * W + w] >> lane) & 1u)) {
      const int r = sh.mr[c];
      ok = r >= 0 && test_bit<W>(anc, r);
    }
    const unsigned ball = __ballot_sync(FULL, ok);
    if (jstar < 0 && ball != 0u) jstar = w * 32 + __ffs(ball) - 1;
  }
  return jstar;
}

// Rotation along the alternating cycle found by warp_back_search (same warp, same lvl, same stamp):
// the row that gives up column jstar takes the column of its successor towards row i, and so on
// down the levels; row i takes jstar. Returns the highest row moved, or -1 on an inconsistency.
template <int NW>
__device__ __forceinline__ int warp_rotate(TeamShared<NW>& sh, const TeamSearchShared<NW>& ts, const int* lvl, int stamp,
                                           int N, int i, int jstar, int lane, int& steps) {
  constexpr int W = NW;
  int cur = MS_AT((int)sh.mr[MS_AT(jstar, N)], N);
  int L = lvl[cur] - stamp;
  int top = i;
  if (L <= 0 || L > N) return -1;
  for (int it = 0; it < N && L > 0; ++it) {
    int cp = -1;
#pragma unroll
    for (int w = 0; w < W; ++w) {
      const int c = w * 32 + lane;
      bool ok = false;
      if (c < N && ((ts.rr[cur * W + w] >> lane) & 1u)) {
        const int r = sh.mr[c];
        ok = r >= 0 && lvl[MS_AT(r, N)] == stamp + L - 1;
      }
      const unsigned ball = __ballot_sync(FULL, ok);
      if (cp < 0 && ball != 0u) cp = w * 32 + __ffs(ball) - 1;
    }
    if (cp < 0) return -1;
    const int nxt = MS_AT((int)sh.mr[cp], N);
    __syncwarp();
    if (lane == 0) { sh.mr[cp] = (short)cur; sh.x[cur] = (short)cp; }
    __syncwarp();
    top = max(top, cur);
    cur = nxt;
    --L;
    ++steps;
  }
  if (cur != i) return -1;
  if (lane == 0) { sh.mr[MS_AT(jstar, N)] = (short)i; sh.x[MS_AT(i, N)] = (short)jstar; }
  __syncwarp();
  return top;
}

// Lexicographically smallest perfect matching of the graph (ts.cc / ts.rr, m.Rr) over the rows
// [start, N), given a perfect matching that already equals the answer below `start`; see
// canonicalise() in common.cuh for the argument. Same result as team_canonicalise. Uniform.
// (For the Birkhoff kernel, whose windows hold one to three rows that could move, this scheme, with
// the search records added, was measured slower than team_canonicalise: 1.85 s against 1.06 s on 256
// matrices of 256 ranks. With nothing to search side by side, one warp working while seven wait is
// worse than eight warps sharing every level. It serves the greedy kernel, where every step
// searches the whole matrix.)
template <int NW>
__device__ __forceinline__ bool team_canonicalise_par(TeamShared<NW>& sh, TeamSearchShared<NW>& ts, TeamRed& red, int N,
                                                      int t, int lane, int warp, bool in, TeamMatch<NW>& m, int& stamp,
                                                      int start, unsigned (&work)[MOESCHED_WORK_FIELDS]) {
  constexpr int W = NW;
  bool ok_all = true;
  bool cand = team_is_candidate<NW>(sh, t, lane, warp, in, m);
  int from = start;
  for (int guard = 0; guard < N; ++guard) {
    unsigned todo[W];
    red.open();
    red.add_member<W>(cand && t >= from, t, lane);
    red.close();
    red.read_set<W>(todo);
    red.next();
    if (!any_bit<W>(todo)) break;
    // a fresh range of level stamps for this round (each warp marks in its own array)
    if (stamp > 0x7f000000) {
      __syncthreads();
#pragma unroll
      for (int w = 0; w < W; ++w) ts.lvl[w][t] = -1;
      stamp = 0;
      __syncthreads();
    }
    stamp += N + 2;
    const int i = kth_member<W>(todo, warp);
    int jstar = -1, levels = 0, reached = 0;
    if (i >= 0) jstar = warp_back_search<NW>(sh, ts, ts.lvl[warp], stamp, N, i, lane, levels, reached);
    if (lane == 0) { ts.res[warp][0] = i; ts.res[warp][1] = jstar; ts.res[warp][2] = levels; ts.res[warp][3] = reached; }
    __syncthreads();
    // results in row order, up to the first row that moves
    int wrot = -1, last_done = from - 1;
    bool bad = false;
    for (int w = 0; w < NW; ++w) {
      const int iw = ts.res[w][0], jw = ts.res[w][1];
      if (iw < 0) break;
      if (jw < 0) { bad = true; break; }
      last_done = iw;
      if (t == 0) { work[WK_SWEEP]++; work[WK_LEVEL] += ts.res[w][2]; work[WK_POP] += ts.res[w][3]; }
      if (jw != sh.x[MS_AT(iw, N)]) { wrot = w; break; }
    }
    if (bad) { ok_all = false; break; }
    from = last_done + 1;
    if (wrot < 0) continue;   // none of the searched rows moves: the matching and the candidates stand
    if (warp == wrot) {
      int steps = 0;
      const int top = warp_rotate<NW>(sh, ts, ts.lvl[warp], stamp, N, ts.res[wrot][0], ts.res[wrot][1], lane, steps);
      if (lane == 0) { sh.misc[4] = top; sh.misc[5] = steps; }
    }
    __syncthreads();
    if (sh.misc[4] < 0) { ok_all = false; break; }
    if (t == 0) work[WK_ROT] += sh.misc[5];
    m.my_x = sh.x[t];
    m.my_mr = sh.mr[t];
    cand = team_is_candidate<NW>(sh, t, lane, warp, in, m);
  }
  return ok_all;
}

}  // namespace moesched
