// Birkhoff-von Neumann decomposition (paper Sec. 3.1), one warp per demand matrix.
//
// The matrix is balanced by north-west-corner padding, then peeled: the support
// graph (positive entries) is kept as one row-set bit mask per column in
// registers; after each subtraction only the rows whose matched entry reached
// zero are re-matched by an augmenting search that disturbs as few low rows as
// possible, and canonicalise() restores the lexicographically smallest perfect
// matching over the window of rows whose column changed (rows before the first
// changed row provably keep theirs; rows after the last one were settled earlier
// and removing edges cannot unsettle them).
#include <atomic>

#include "common.cuh"

namespace moesched {

// MODE 0: matrix in this CTA's shared memory; 1: split over a 2-CTA cluster; 2: working copy
// in global memory (scratch), which leaves room for many more warps per SM.
// COUNT: the per-matrix work counters are wanted (they are plain register increments that the
// compiler drops, registers included, when nothing reads them).
//
// PACE. The warp schedulers of an SM serve their resident warps in a fixed order of preference. With several
// equally long decompositions per scheduler the preferred warps run at full speed and finish early, and the
// others are left to finish alone, each stalled on its own dependent chain with most issue slots empty
// (measured, N = 64, B = 4096, all warps resident from the start: the warps in the first four slots of an SM
// finish after 22.7 ms, those in the last four after 39.3 ms). When the whole batch is resident at once the
// launcher therefore switches pacing on: every warp publishes, every PACE_EVERY matchings, how many entries its
// matrix has left, reads the figures of the warps that share its scheduler (warp slot modulo 4), and sleeps for a
// moment when it is well ahead of the slowest of them. The slots go to the warps behind and all finish together
// (40.5 -> 38.9 ms). A sleep is a plain delay, never a wait for another warp: results and termination do not
// depend on it. Entries carry the launch's number, so figures left by another launch are ignored.
constexpr int PACE_EVERY = 16;          // matchings between two looks (a power of two)
constexpr unsigned PACE_SLACK = 32;     // entries a warp may be ahead before it sleeps
constexpr unsigned PACE_NS_PER_ENTRY = 2000, PACE_NS_MAX = 200000;
__device__ unsigned long long g_pace[256][64];   // [SM][warp slot] = launch number << 32 | entries left

template <int CPL, int MODE, bool COUNT, bool PACE = false>
__global__ void __launch_bounds__(128, CPL <= 2 ? 7 : 0) bvn_kernel(int B, int N, int S, const int32_t* __restrict__ demand, int k_max,
                                                  uint8_t* __restrict__ perm, int32_t* __restrict__ coef,
                                                  int32_t* __restrict__ count, int32_t* __restrict__ aug,
                                                  int32_t* scratch, int32_t* __restrict__ status,
                                                  long long* __restrict__ work_out, unsigned pace_launch = 0u) {
  constexpr int W = CPL;
  constexpr bool CLUSTER = MODE == 1;
  constexpr bool USE_MEMO = true;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  WarpCtx cx;
  if constexpr (MODE == 2) cx = warp_prologue_global<CPL>(B, N, S, demand, scratch, smem_raw);
  else cx = warp_prologue<CPL, CLUSTER>(B, N, S, demand, smem_raw);
  if (!cx.worker) { cluster_epilogue<CLUSTER>(); return; }
  const int lane = cx.lane, b = cx.b;
  const MatView A = cx.M;
  short* x = cx.x;
  unsigned* hist = cx.hist;
  const bool loaded = cx.loaded;

  unsigned work[MOESCHED_WORK_FIELDS];
#pragma unroll
  for (int q = 0; q < MOESCHED_WORK_FIELDS; ++q) work[q] = 0u;

  const bool lane_in = lane * CPL < S;
  int st_code = loaded ? MOESCHED_ST_OK : MOESCHED_ST_INTERNAL;
  int k = 0;

  // ---- column sums (registers), row sums (one reduction per row), validation ----
  long long csum[CPL];
#pragma unroll
  for (int s = 0; s < CPL; ++s) csum[s] = 0;
  long long rsum_mine[CPL];   // row sums of the rows lane*CPL+s
#pragma unroll
  for (int s = 0; s < CPL; ++s) rsum_mine[s] = 0;
  int neg = 0;
  for (int r = 0; r < N; ++r) {
    long long part = 0;
    if (lane_in) {
      RowVec<CPL> rv = load_cols<CPL>(A.row(r), lane);
#pragma unroll
      for (int s = 0; s < CPL; ++s) {
        if (lane * CPL + s < N) {
          neg |= rv.v[s] < 0;
          csum[s] += rv.v[s];
          part += rv.v[s];
        }
      }
    }
    // 64-bit warp sum
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(FULL, part, o);
    if (lane == r / CPL) put<CPL>(rsum_mine, r % CPL, part);
  }
  neg = __any_sync(FULL, neg);
  long long T = 0;
#pragma unroll
  for (int s = 0; s < CPL; ++s) T = max(T, max(csum[s], rsum_mine[s]));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) T = max(T, __shfl_xor_sync(FULL, T, o));
  if (st_code == MOESCHED_ST_OK && (neg || T > 2147483647LL)) st_code = MOESCHED_ST_BAD_INPUT;

  if (st_code == MOESCHED_ST_OK) {
    // ---- north-west-corner fill of the deficits: lowest row first, then lowest column ----
    // The staircase visits at most 2N-1 cells; row and column deficits are fetched by shuffle.
    {
      int i = 0, j = 0;
      long long a = 0, bb = 0;
      bool have_a = false, have_b = false;
      for (int it = 0; it < 4 * N + 4 && i < N && j < N; ++it) {
        if (!have_a) { a = T - __shfl_sync(FULL, pick<CPL>(rsum_mine, i % CPL), i / CPL); have_a = true; }
        if (!have_b) { bb = T - __shfl_sync(FULL, pick<CPL>(csum, j % CPL), j / CPL); have_b = true; }
        if (a == 0) { ++i; have_a = false; continue; }
        if (bb == 0) { ++j; have_b = false; continue; }
        const long long e = min(a, bb);
        if (lane == 0) A.row(i)[j] += (int)e;
        a -= e;
        bb -= e;
      }
      __syncwarp();
    }
    if (aug != nullptr) {
      int32_t* ao = aug + (size_t)b * N * N;
      for (int r = 0; r < N; ++r) {
        const int* rp = A.row(r);
        for (int c = lane; c < N; c += 32) ao[(size_t)r * N + c] = rp[c];
      }
    }

    // ---- support graph: C[s] = rows with a positive entry in the lane's column s ----
    unsigned C[CPL][CPL];
#pragma unroll
    for (int s = 0; s < CPL; ++s)
#pragma unroll
      for (int w = 0; w < W; ++w) C[s][w] = 0u;
    int nnz = 0;
#pragma unroll
    for (int w = 0; w < W; ++w) {
      for (int q = 0; q < 32; ++q) {
        const int r = w * 32 + q;
        if (r >= N) break;
        if (lane_in) {
          RowVec<CPL> rv = load_cols<CPL>(A.row(r), lane);
#pragma unroll
          for (int s = 0; s < CPL; ++s)
            if (lane * CPL + s < N && rv.v[s] > 0) { C[s][w] |= 1u << q; ++nnz; }
        }
      }
    }
    nnz = __reduce_add_sync(FULL, nnz);

    Match<CPL> M;
    M.reset();
    CanonMemo<CPL> memo;
    memo.reset();
    for (int q = lane; q < N * W; q += 32) hist[(N + 1) * W + q] = 0u;   // per-row memo starts empty
    for (int r = lane; r < N; r += 32) x[r] = -1;
    __syncwarp();

    uint8_t* pout = perm + (size_t)b * k_max * N;
    int32_t* cout_ = coef + (size_t)b * k_max;
    int lo_changed = 0, hi_changed = N - 1;   // window of rows whose column may not be final
    unsigned freerows[W];   // uniform: rows without a column
#pragma unroll
    for (int w = 0; w < W; ++w) {
      const int lo = w * 32;
      freerows[w] = N >= lo + 32 ? 0xffffffffu : (N <= lo ? 0u : (0xffffffffu >> (lo + 32 - N)));
    }

    unsigned pace_seen = 0u;   // the largest figure seen at the last look
    while (nnz > 0 && k < k_max) {
      if constexpr (PACE) {
        if ((k & (PACE_EVERY - 1)) == 0) {
          unsigned pace_sm, pace_slot;   // read afresh every time rather than kept in registers across the loop
          asm volatile("mov.u32 %0, %%smid;" : "=r"(pace_sm));
          asm volatile("mov.u32 %0, %%warpid;" : "=r"(pace_slot));
          pace_sm &= 255u;
          pace_slot &= 63u;
          if (lane == 0) g_pace[pace_sm][pace_slot] = ((unsigned long long)pace_launch << 32) | (unsigned)nnz;
          unsigned left = 0u;
          if (lane < 16) {
            const unsigned long long v =
                *reinterpret_cast<const volatile unsigned long long*>(&g_pace[pace_sm][(pace_slot & 3u) + 4u * lane]);
            if ((unsigned)(v >> 32) == pace_launch) left = (unsigned)v;
          }
          left = __reduce_max_sync(FULL, left);   // the most entries left among the warps of this scheduler
          // (a figure that has not moved since the last look is not slept on twice: an entry orphaned by a warp
          // whose slot changed under preemption must not hold the others back)
          if (left > (unsigned)nnz + PACE_SLACK && left != pace_seen)
            __nanosleep(min((left - (unsigned)nnz - PACE_SLACK) * PACE_NS_PER_ENTRY, PACE_NS_MAX));
          pace_seen = left;
        }
      }
      // re-match the free rows: a single row that lost its entry is re-matched canonically at once
      bool okm = true;
      if (k > 0) {
        // rows that lost their entry are re-matched canonically, lowest first, as long as that works
        for (int it = 0; it < N; ++it) {
          const int r0 = lowest_bit<W>(freerows);
          if (r0 < 0) break;
          int single = 0;
#pragma unroll
          for (int w = 0; w < W; ++w) single += __popc(freerows[w]);
          const int rc = canonical_repair<CPL>(N, lane, r0, C, M, x, hist, hi_changed, memo.changed, work, single == 1,
                                               lo_changed);
          if (rc < 0) { okm = false; break; }
          if (rc == 0) { work[WK_BATCH]++; break; }   // needs rows below r0: the general search below takes over
          clear_bit<W>(freerows, r0);
          if (rc == 2) { work[WK_BATCH]++; break; }   // rows below r0 had to move: the window starts at the lowest of them
          work[WK_TIGHT]++;
          lo_changed = min(lo_changed, r0 + 1);   // row r0 has its final column; the rows that moved lie above it
        }
        if (!okm) { st_code = MOESCHED_ST_INTERNAL; break; }
      }
      for (int it = 0; it < N; ++it) {
        const int f = lowest_bit<W>(freerows);
        if (f < 0) break;
        if (!augment_from<CPL>(N, lane, f, C, M, x, lo_changed, hi_changed, memo.changed, work)) { okm = false; break; }
        clear_bit<W>(freerows, f);
      }
      if (!okm || any_bit<W>(freerows)) { st_code = MOESCHED_ST_INTERNAL; break; }
      work[WK_SKIP] += lo_changed;
      if (!canonicalise<CPL, USE_MEMO>(N, lane, lo_changed, hi_changed, C, M, x, hist, memo, work)) {
        st_code = MOESCHED_ST_INTERNAL;
        break;
      }

      // coefficient = smallest matched entry; subtract it along the matching
      int val[CPL], cmin = INF32;
      int* cell[CPL];   // the lane's matched entries
#pragma unroll
      for (int s = 0; s < CPL; ++s) {
        const int c = lane * CPL + s;
        val[s] = INF32;
        cell[s] = nullptr;
        if (c < N) {
          // with the working copy in global memory every row is "near": no split to test
          const int mrow = MS_AT(M.mr[s], N);
          cell[s] = (MODE == 2 ? A.near_ + (size_t)mrow * A.S : A.row(mrow)) + c;
          val[s] = *cell[s];
          cmin = min(cmin, val[s]);
        }
      }
      cmin = __reduce_min_sync(FULL, cmin);
      lo_changed = N;
      hi_changed = -1;
      unsigned gone[W];
#pragma unroll
      for (int w = 0; w < W; ++w) gone[w] = 0u;
      int zeroed = 0;
#pragma unroll
      for (int s = 0; s < CPL; ++s) {
        const int c = lane * CPL + s;
        if (c < N) {
          const int nv = val[s] - cmin;
          *cell[s] = nv;
          if (nv == 0) {
#pragma unroll
            for (int w = 0; w < W; ++w) C[s][w] &= ~M.word(s, w);
            M.add_to(gone, s);
            ++zeroed;
          }
        }
      }
      for (int r = lane; r < N; r += 32) pout[(size_t)k * N + r] = (uint8_t)x[r];
      if (lane == 0) cout_[k] = cmin;
      ++k;
      work[WK_MATCH]++;
      nnz -= __reduce_add_sync(FULL, zeroed);
#pragma unroll
      for (int w = 0; w < W; ++w) freerows[w] = __reduce_or_sync(FULL, gone[w]);
      // unmatch the rows whose entry vanished
      M.release(freerows);
      // (x[r] was last read, for the permutation row above, by the lane that clears it here; the barrier after the
      // loop makes the cleared entries visible to the other lanes, whose later updates of x are made by every lane)
#pragma unroll
      for (int q = 0; q < W; ++q) {   // lane l looks after rows l, l + 32, ...
        const int r = q * 32 + lane;
        if (r < N && ((freerows[q] >> lane) & 1u)) x[r] = -1;
      }
      __syncwarp();
    }
    if (st_code == MOESCHED_ST_OK && nnz > 0) st_code = MOESCHED_ST_TRUNCATED;
  }

  if (st_code == MOESCHED_ST_BAD_INPUT) k = 0;
  if constexpr (PACE) {   // this warp no longer counts (it may have moved on without entering the loop)
    unsigned sm, slot;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
    asm volatile("mov.u32 %0, %%warpid;" : "=r"(slot));
    if (lane == 0) g_pace[sm & 255u][slot & 63u] = 0ull;
  }
  if (lane == 0) {
    count[b] = k;
    status[b] = st_code;
  }
  if constexpr (COUNT) {
    if (work_out != nullptr && lane == 0) {
#pragma unroll
      for (int q = 0; q < MOESCHED_WORK_FIELDS; ++q) work_out[(size_t)b * MOESCHED_WORK_FIELDS + q] = work[q];
    }
  }
  cluster_epilogue<CLUSTER>();
}

// ---- host side ---------------------------------------------------------------------------

// Number of this paced launch (never 0; entries of the pacing table with another number are ignored).
static unsigned next_pace_launch() {
  static std::atomic<unsigned> n{0u};
  unsigned v = ++n;
  if (v == 0u) v = ++n;
  return v;
}

cudaError_t run_bvn(int B, int N, const int32_t* demand, int k_max, uint8_t* perm, int32_t* coef, int32_t* count,
                    int32_t* aug, int32_t* scratch, int32_t* status, long long* work, cudaStream_t stream) {
  Geometry ge = plan_geometry(N);
#define MOESCHED_GO(C, M)                                                                                     \
  do {                                                                                                        \
    if (work != nullptr)                                                                                      \
      return launch_warp_kernel(bvn_kernel<C, M, true>, ge, B, stream, B, N, ge.S, demand, k_max, perm, coef, \
                                count, aug, scratch, status, work, 0u);                                       \
    return launch_warp_kernel(bvn_kernel<C, M, false>, ge, B, stream, B, N, ge.S, demand, k_max, perm, coef,  \
                              count, aug, scratch, status, work, 0u);                                         \
  } while (0)
  // Above 128 ranks a batch that leaves most SMs with a single warp goes to the kernel that puts a
  // CTA of eight warps on each matrix (measured at N = 256, B = 256: 1.0 s against 1.8 s; at N = 128,
  // B = 1024 one warp per matrix is the faster of the two, 0.32 s against 0.46 s).
  if (scratch != nullptr && N > 128 && B < 8 * sm_count())
    return run_bvn_team(B, N, demand, k_max, perm, coef, count, aug, scratch, status, work, stream);
  if (scratch != nullptr) {
    // working copy in global memory: four matrices per CTA, shared memory only for hist and x
    ge.cluster = false;
    ge.S = bvn_scratch_stride(N);
    // four matrices per CTA once there are enough of them to give every SM several CTAs;
    // a small batch is spread one matrix per CTA so that no SM sits idle
    ge.wpb = B >= 16 * sm_count() ? 4 : 1;
    ge.smem = warp_smem_bytes_global(N, ge.cpl) * ge.wpb;
    // pacing (see PACE above) when every scheduler gets three warps or more and the whole batch is resident at once
    if (work == nullptr && B >= 12 * sm_count()) {
#define MOESCHED_PACED(C)                                                                                          \
  do {                                                                                                             \
    int per_sm = 0;                                                                                                \
    auto kern = bvn_kernel<C, 2, false, true>;                                                                     \
    cudaError_t eo = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ge.smem);        \
    if (eo == cudaSuccess) eo = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, 32 * ge.wpb, ge.smem); \
    if (eo != cudaSuccess) return eo;                                                                              \
    if ((long long)per_sm * sm_count() >= (B + ge.wpb - 1) / ge.wpb)                                               \
      return launch_warp_kernel(kern, ge, B, stream, B, N, ge.S, demand, k_max, perm, coef, count, aug, scratch,   \
                                status, work, next_pace_launch());                                                 \
  } while (0)
      switch (ge.cpl) {
        case 1: MOESCHED_PACED(1); break;
        case 2: MOESCHED_PACED(2); break;
        case 4: MOESCHED_PACED(4); break;
        default: MOESCHED_PACED(8); break;
      }
#undef MOESCHED_PACED
    }
    switch (ge.cpl) {
      case 1: MOESCHED_GO(1, 2);
      case 2: MOESCHED_GO(2, 2);
      case 4: MOESCHED_GO(4, 2);
      default: MOESCHED_GO(8, 2);
    }
  }
  if (ge.cluster) MOESCHED_GO(8, 1);
  switch (ge.cpl) {
    case 1: MOESCHED_GO(1, 0);
    case 2: MOESCHED_GO(2, 0);
    case 4: MOESCHED_GO(4, 0);
    default: MOESCHED_GO(8, 0);
  }
#undef MOESCHED_GO
}

}  // namespace moesched
