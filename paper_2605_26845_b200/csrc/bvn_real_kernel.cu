// Birkhoff-von Neumann decomposition of a REAL-valued matrix (paper Sec. 3.1: A = sum_k lambda_k P_k
// for a doubly stochastic A, as obtained from Sinkhorn-Knopp scaling), one warp per matrix.
//
// The combinatorial part is the one of bvn_kernel.cu (support graph as bit masks in registers,
// re-matching of the rows whose entry vanished, canonicalise() over the window of changed rows);
// only the entries are doubles, held in a global working copy. Every arithmetic step is one exact
// IEEE operation (a minimum, a subtraction, a comparison with the tolerance) taken in a fixed
// order, so the result is reproducible bit for bit. A scaled matrix is doubly stochastic only up
// to the error of its last sweep: when the support has no perfect matching left the decomposition
// stops and reports what remains.
#include "common.cuh"

namespace moesched {

namespace {

__device__ __forceinline__ double warp_min_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmin(v, __shfl_xor_sync(FULL, v, o));
  return v;
}
__device__ __forceinline__ double warp_max_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(FULL, v, o));
  return v;
}

}  // namespace

template <int CPL>
__global__ void __launch_bounds__(128) bvn_real_kernel(int B, int N, int S, const double* __restrict__ matrix, double tol,
                                                       int k_max, uint8_t* __restrict__ perm,
                                                       double* __restrict__ lambda, int32_t* __restrict__ count,
                                                       double* __restrict__ sum_lambda, double* __restrict__ max_left,
                                                       double* scratch, int32_t* __restrict__ status) {
  constexpr int W = CPL;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int b = blockIdx.x * (blockDim.x >> 5) + warp;
  if (b >= B) return;
  unsigned char* base = smem_raw + (size_t)warp * warp_smem_bytes_global(N, CPL);
  unsigned* hist = reinterpret_cast<unsigned*>(base);
  short* x = reinterpret_cast<short*>(base + hist_bytes_for(N, CPL));
  double* A = scratch + (size_t)b * N * S;
  const double* src = matrix + (size_t)b * N * N;

  unsigned work[MOESCHED_WORK_FIELDS];
#pragma unroll
  for (int q = 0; q < MOESCHED_WORK_FIELDS; ++q) work[q] = 0u;

  // ---- working copy: entries at or below the tolerance are dropped; negative or NaN entries reject ----
  int bad = 0;
  for (int r = 0; r < N; ++r)
    for (int c = lane; c < S; c += 32) {
      double v = 0.0;
      if (c < N) {
        v = src[(size_t)r * N + c];
        bad |= !(v >= 0.0);
        if (!(v > tol)) v = 0.0;
      }
      A[(size_t)r * S + c] = v;
    }
  bad = __any_sync(FULL, bad);
  __syncwarp();

  int st_code = bad ? MOESCHED_ST_BAD_INPUT : MOESCHED_ST_OK;
  int k = 0;
  double total = 0.0;

  if (st_code == MOESCHED_ST_OK) {
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
#pragma unroll
        for (int s = 0; s < CPL; ++s) {
          const int c = lane * CPL + s;
          if (c < N && A[(size_t)r * S + c] > 0.0) { C[s][w] |= 1u << q; ++nnz; }
        }
      }
    }
    nnz = __reduce_add_sync(FULL, nnz);

    Match<CPL> M;
    M.reset();
    CanonMemo<CPL> memo;
    memo.reset();
    for (int q = lane; q < N * W; q += 32) hist[(N + 1) * W + q] = 0u;
    for (int r = lane; r < N; r += 32) x[r] = -1;
    __syncwarp();

    uint8_t* pout = perm + (size_t)b * k_max * N;
    double* lout = lambda + (size_t)b * k_max;
    int lo_changed = 0, hi_changed = N - 1;
    unsigned freerows[W];
#pragma unroll
    for (int w = 0; w < W; ++w) {
      const int lo = w * 32;
      freerows[w] = N >= lo + 32 ? 0xffffffffu : (N <= lo ? 0u : (0xffffffffu >> (lo + 32 - N)));
    }

    bool exhausted = false;   // the support has no perfect matching any more
    while (nnz > 0 && k < k_max) {
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
      if (!okm) { exhausted = true; break; }
      if (!canonicalise<CPL, true>(N, lane, lo_changed, hi_changed, C, M, x, hist, memo, work)) {
        st_code = MOESCHED_ST_INTERNAL;
        break;
      }
      // lambda = smallest matched entry; subtract it along the matching; what falls to the tolerance vanishes
      double val[CPL], cmin = 1e300;
#pragma unroll
      for (int s = 0; s < CPL; ++s) {
        const int c = lane * CPL + s;
        val[s] = 1e300;
        if (c < N) {
          val[s] = A[(size_t)MS_AT(M.mr[s], N) * S + c];
          cmin = fmin(cmin, val[s]);
        }
      }
      cmin = warp_min_f64(cmin);
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
          double nv = __dsub_rn(val[s], cmin);
          if (!(nv > tol)) nv = 0.0;
          A[(size_t)MS_AT(M.mr[s], N) * S + c] = nv;
          if (nv == 0.0) {
#pragma unroll
            for (int w = 0; w < W; ++w) C[s][w] &= ~M.word(s, w);
            M.add_to(gone, s);
            ++zeroed;
          }
        }
      }
      for (int r = lane; r < N; r += 32) pout[(size_t)k * N + r] = (uint8_t)x[r];
      if (lane == 0) lout[k] = cmin;
      total = __dadd_rn(total, cmin);
      ++k;
      nnz -= __reduce_add_sync(FULL, zeroed);
#pragma unroll
      for (int w = 0; w < W; ++w) freerows[w] = __reduce_or_sync(FULL, gone[w]);
      M.release(freerows);
      // (x[r] was last read, for the permutation row above, by the lane that clears it here; the barrier after the
      // loop makes the cleared entries visible to the other lanes, whose later updates of x are made by every lane)
#pragma unroll
      for (int q = 0; q < W; ++q) {
        const int r = q * 32 + lane;
        if (r < N && ((freerows[q] >> lane) & 1u)) x[r] = -1;
      }
      __syncwarp();
    }
    if (st_code == MOESCHED_ST_OK && (nnz > 0 || exhausted)) st_code = MOESCHED_ST_TRUNCATED;
  }

  double left = 0.0;
  if (st_code != MOESCHED_ST_BAD_INPUT) {
    __syncwarp();
    for (int r = 0; r < N; ++r)
      for (int c = lane; c < N; c += 32) left = fmax(left, A[(size_t)r * S + c]);
    left = warp_max_f64(left);
  } else {
    k = 0;
  }
  if (lane == 0) {
    count[b] = k;
    status[b] = st_code;
    sum_lambda[b] = st_code == MOESCHED_ST_BAD_INPUT ? 0.0 : total;
    max_left[b] = left;
  }
}

cudaError_t run_bvn_real(int B, int N, const double* matrix, double tol, int k_max, uint8_t* perm, double* lambda,
                         int32_t* count, double* sum_lambda, double* max_left, double* scratch, int32_t* status,
                         cudaStream_t stream) {
  Geometry ge = plan_geometry(N);
  ge.cluster = false;
  ge.S = bvn_scratch_stride(N);
  ge.wpb = B >= 16 * sm_count() ? 4 : 1;
  ge.smem = warp_smem_bytes_global(N, ge.cpl) * ge.wpb;
#define MOESCHED_GO(C)                                                                                              \
  return launch_warp_kernel(bvn_real_kernel<C>, ge, B, stream, B, N, ge.S, matrix, tol, k_max, perm, lambda, count, \
                            sum_lambda, max_left, scratch, status)
  switch (ge.cpl) {
    case 1: MOESCHED_GO(1);
    case 2: MOESCHED_GO(2);
    case 4: MOESCHED_GO(4);
    default: MOESCHED_GO(8);
  }
#undef MOESCHED_GO
}

}  // namespace moesched
