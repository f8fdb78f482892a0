// Sinkhorn-Knopp scaling (the preprocessing paper Sec. 3.1 names for the Birkhoff-von Neumann
// decomposition), one warp per demand matrix, IEEE double throughout.
//
// X = D + smooth; one sweep divides every entry by the sum of its row, then every entry by the sum
// of its column (IEEE division, correctly rounded). The sums are defined left to right (rows) and top to bottom
// (columns) with one rounding per operation, so that the result does not depend on how the work
// is spread over lanes:
//   * a column sum is accumulated by the lane that owns the column (column c: lane c % 32) while
//     the warp walks the rows from the top -- coalesced loads, sequential order;
//   * a row sum is accumulated by the lane that owns the row of the current block of 32 rows: the
//     warp loads 32 x 32 tiles with coalesced row loads into shared memory (row stride 33, no
//     bank conflicts) and every lane then adds its row's 32 entries in order.
// Up to N = 64 the matrix stays in shared memory for the whole call (32 KB of doubles per warp) and
// global memory sees the demand once on the way in and the results once on the way out; above
// that it lives in the caller's `scaled` buffer (global memory, L2-resident while a matrix is
// worked on). The pending column scaling of one pass is applied while the next pass reads the matrix,
// so that a sweep costs two reads and two writes of the matrix. Every arithmetic step uses the
// round-to-nearest intrinsics, which also keeps the compiler from fusing multiplies and adds.
#include "common.cuh"

namespace moesched {

namespace {

constexpr int SK_TILE = 32 * 33;          // doubles of the tile
constexpr int SK_WARP = SK_TILE + 256;    // plus one row sum per row

// Applies the pending column scaling (entry (r, c) divided by col_div of its column) if HAVE_MUL, writes
// the scaled entries back, and leaves in rsum[r] (shared memory) the sum of row r, left to right.
template <int CPL, bool HAVE_MUL>
__device__ __forceinline__ void row_sums_pass(int N, int lane, double* S, double* tile, const double (&col_div)[CPL],
                                              double* rsum) {
  for (int rb = 0; rb * 32 < N; ++rb) {
    double acc = 0.0;
#pragma unroll
    for (int cb = 0; cb < CPL; ++cb) {
      if (cb * 32 < N) {
        const int c = cb * 32 + lane;
        for (int rr = 0; rr < 32; ++rr) {
          const int r = rb * 32 + rr;
          double v = 0.0;
          if (r < N && c < N) {
            v = S[(size_t)r * N + c];
            if (HAVE_MUL) {
              v = __ddiv_rn(v, col_div[cb]);
              S[(size_t)r * N + c] = v;
            }
          }
          tile[rr * 33 + lane] = v;
        }
        __syncwarp();
        const int lim = min(32, N - cb * 32);
        for (int cc = 0; cc < lim; ++cc) acc = __dadd_rn(acc, tile[lane * 33 + cc]);
        __syncwarp();
      }
    }
    if (rb * 32 + lane < N) rsum[rb * 32 + lane] = acc;
  }
  __syncwarp();
}

}  // namespace

template <int CPL, bool RESIDENT>
__global__ void __launch_bounds__(128) sinkhorn_kernel(int B, int N, const int32_t* __restrict__ demand, int iters,
                                                       double smooth, double scale, double* __restrict__ scaled,
                                                       int32_t* __restrict__ fixed, double* __restrict__ stretch,
                                                       double* __restrict__ row_err, int32_t* __restrict__ status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int b = blockIdx.x * (blockDim.x >> 5) + warp;
  if (b >= B) return;
  double* tile = reinterpret_cast<double*>(smem_raw) + (size_t)warp * SK_WARP;
  double* rsum = tile + SK_TILE;
  const int32_t* D = demand + (size_t)b * N * N;
  double* Sout = scaled + (size_t)b * N * N;
  double* S = RESIDENT ? reinterpret_cast<double*>(smem_raw) + (size_t)(blockDim.x >> 5) * SK_WARP + (size_t)warp * N * N
                       : Sout;
  int32_t* Q = fixed + (size_t)b * N * N;

  int bad = 0;
  for (int e = lane; e < N * N; e += 32) {
    const int d = D[e];
    bad |= d < 0;
    S[e] = __dadd_rn((double)d, smooth);
  }
  bad = __any_sync(FULL, bad);
  __syncwarp();

  double col_div[CPL];   // column sums of the last column pass: the division by them is still pending
#pragma unroll
  for (int s = 0; s < CPL; ++s) col_div[s] = 1.0;
  for (int it = 0; it < iters && !bad; ++it) {
    if (it == 0) row_sums_pass<CPL, false>(N, lane, S, tile, col_div, rsum);
    else row_sums_pass<CPL, true>(N, lane, S, tile, col_div, rsum);
    // a row without mass cannot be scaled
    int zero = 0;
    for (int r = lane; r < N; r += 32) zero |= !(rsum[r] > 0.0);
    if (__any_sync(FULL, zero)) { bad = 1; break; }
    // divide the rows by their sums and accumulate the column sums from the top
    double csum[CPL];
#pragma unroll
    for (int s = 0; s < CPL; ++s) csum[s] = 0.0;
    for (int r = 0; r < N; ++r) {
      const double rv = rsum[r];
#pragma unroll
      for (int s = 0; s < CPL; ++s) {
        const int c = s * 32 + lane;
        if (c < N) {
          const double v = __ddiv_rn(S[(size_t)r * N + c], rv);
          S[(size_t)r * N + c] = v;
          csum[s] = __dadd_rn(csum[s], v);
        }
      }
    }
    zero = 0;
#pragma unroll
    for (int s = 0; s < CPL; ++s) {
      if (s * 32 + lane < N) zero |= !(csum[s] > 0.0);
      col_div[s] = csum[s];
    }
    if (__any_sync(FULL, zero)) { bad = 1; break; }
    __syncwarp();
  }

  if (bad) {
    __syncwarp();
    for (int e = lane; e < N * N; e += 32) { Sout[e] = 0.0; Q[e] = 0; }
    if (lane == 0) { stretch[b] = 0.0; row_err[b] = 0.0; status[b] = MOESCHED_ST_BAD_INPUT; }
    return;
  }

  // the last column scaling, the row sums of the result, the fixed-point matrix and the stretch
  row_sums_pass<CPL, true>(N, lane, S, tile, col_div, rsum);
  double err = 0.0;
  for (int r = lane; r < N; r += 32) err = fmax(err, fabs(__dadd_rn(rsum[r], -1.0)));
  __syncwarp();
  double st = 0.0;
  int dropped = 0;
  for (int e = lane; e < N * N; e += 32) {
    const double v = S[e];
    if (RESIDENT) Sout[e] = v;
    const double q = floor(__dadd_rn(__dmul_rn(v, scale), 0.5));
    const int qi = (int)q;
    Q[e] = qi;
    const int d = D[e];
    if (d > 0) {
      if (qi > 0) st = fmax(st, __ddiv_rn(__dmul_rn((double)d, scale), (double)qi));
      else dropped = 1;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    err = fmax(err, __shfl_xor_sync(FULL, err, o));
    st = fmax(st, __shfl_xor_sync(FULL, st, o));
  }
  dropped = __any_sync(FULL, dropped);
  if (lane == 0) {
    stretch[b] = st;
    row_err[b] = err;
    status[b] = dropped ? MOESCHED_ST_TRUNCATED : MOESCHED_ST_OK;
  }
}

__global__ void __launch_bounds__(256) sinkhorn_durations_kernel(int B, int k_stride, const int32_t* __restrict__ coef,
                                                                 const int32_t* __restrict__ count,
                                                                 const double* __restrict__ stretch, double scale,
                                                                 int32_t* __restrict__ dur) {
  const int b = blockIdx.y;
  if (b >= B) return;
  const int K = min(max(count[b], 0), k_stride);
  const double st = stretch[b];
  for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < K; k += gridDim.x * blockDim.x) {
    const double x = __dmul_rn((double)coef[(size_t)b * k_stride + k], st);
    const double d = ceil(__ddiv_rn(x, scale));
    dur[(size_t)b * k_stride + k] = d >= 2147483647.0 ? 2147483647 : (d > 0.0 ? (int)d : 0);
  }
}

// ---- host side ---------------------------------------------------------------------------

cudaError_t run_sinkhorn(int B, int N, const int32_t* demand, int iters, double smooth, int scale_bits,
                         double* scaled, int32_t* fixed, double* stretch, double* row_err, int32_t* status,
                         cudaStream_t stream) {
  const bool resident = N <= 64;
  const int wpb = resident ? 1 : 4;
  const size_t smem = (size_t)wpb * (SK_WARP + (resident ? N * N : 0)) * sizeof(double);
  const double scale = (double)(1 << scale_bits);
  const int grid = (B + wpb - 1) / wpb;
#define MOESCHED_GO(C, R)                                                                                           \
  do {                                                                                                              \
    cudaError_t e = cudaFuncSetAttribute(sinkhorn_kernel<C, R>, cudaFuncAttributeMaxDynamicSharedMemorySize,        \
                                         (int)smem);                                                                \
    if (e != cudaSuccess) return e;                                                                                 \
    sinkhorn_kernel<C, R><<<grid, 32 * wpb, smem, stream>>>(B, N, demand, iters, smooth, scale, scaled, fixed,      \
                                                            stretch, row_err, status);                              \
    return cudaGetLastError();                                                                                      \
  } while (0)
  if (N <= 32) MOESCHED_GO(1, true);
  if (N <= 64) MOESCHED_GO(2, true);
  if (N <= 128) MOESCHED_GO(4, false);
  MOESCHED_GO(8, false);
#undef MOESCHED_GO
}

cudaError_t run_sinkhorn_durations(int B, int k_stride, const int32_t* coef, const int32_t* count,
                                   const double* stretch, int scale_bits, int32_t* dur, cudaStream_t stream) {
  const double scale = (double)(1 << scale_bits);
  // B up to 65535 rows of the grid per launch
  for (int b0 = 0; b0 < B; b0 += 65535) {
    const int nb = min(65535, B - b0);
    dim3 grid((k_stride + 255) / 256 > 64 ? 64 : (k_stride + 255) / 256, nb);
    sinkhorn_durations_kernel<<<grid, 256, 0, stream>>>(nb, k_stride, coef + (size_t)b0 * k_stride, count + b0,
                                                        stretch + b0, scale, dur + (size_t)b0 * k_stride);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace moesched
