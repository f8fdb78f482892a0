// Device-side building blocks shared by the kernels in which one warp owns one
// demand matrix: the matrix is held in shared memory (as int32 above 232 ranks it
// is spread over the two CTAs of a thread-block cluster) or in a global working
// copy, and the matching state lives in registers.
//
// Ownership: lane l owns columns (and rows, where a per-row value is kept in
// registers) l*CPL .. l*CPL+CPL-1, CPL = 1, 2, 4 or 8, so that a row scan is one
// vector load per lane. Sets of rows or columns are bit masks of W = CPL 32-bit
// words; masks that every lane holds identically are "uniform".
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/moesched.h"

namespace moesched {

constexpr unsigned FULL = 0xffffffffu;
constexpr int INF32 = 0x7fffffff;

// Index checks of the debug build (-DMOESCHED_CHECKED; the stand-in for a memory checker on machines
// where none can be run): every shared- or global-memory index that comes out of the matching state
// (a matched row or column, a path predecessor, a search level) goes through MS_AT(index, limit).
// In the checked build an index outside [0, limit) is counted in a per-file device counter and
// replaced by 0, so that the access stays in bounds and the kernel ends normally; the host reads the sum
// of the counters through moesched_debug_index_faults(). In the normal build MS_AT(i, n) is just (i).
#ifdef MOESCHED_CHECKED
static __device__ unsigned g_index_faults;
__device__ __forceinline__ int checked_index(int i, int n) {
  if ((unsigned)i >= (unsigned)n) {
    atomicAdd(&g_index_faults, 1u);
    return 0;
  }
  return i;
}
#define MS_AT(i, n) ::moesched::checked_index((i), (n))
using FaultReader = unsigned (*)();
void register_fault_reader(FaultReader reader);   // api.cu
static unsigned read_faults_of_this_file() {
  unsigned v = 0;
  if (cudaMemcpyFromSymbol(&v, g_index_faults, sizeof v) != cudaSuccess) return 0xffffffffu;
  return v;
}
static const bool g_fault_reader_registered = (register_fault_reader(&read_faults_of_this_file), true);
#else
#define MS_AT(i, n) (i)
#endif

enum WorkField { WK_SCAN = 0, WK_AUG = 1, WK_TIGHT = 2, WK_SWEEP = 3, WK_LEVEL = 4, WK_ROT = 5, WK_MATCH = 6, WK_SKIP = 7, WK_POP = 8, WK_BATCH = 9 };

// ---- small helpers on register arrays -------------------------------------------------

// Bit access with a run-time index is written as arithmetic over ALL words (never as
// "touch word k if idx/32 == k"), so that the compiler cannot turn it into an indexed
// access that would push the register array into local memory.
// (Two-word masks take a 64-bit path: one wide shift instead of per-word selects.)
__device__ __forceinline__ unsigned long long as64(const unsigned (&m)[2]) {
  return ((unsigned long long)m[1] << 32) | m[0];
}
template <int W>
__device__ __forceinline__ bool test_bit(const unsigned (&m)[W], int idx) {
  if constexpr (W == 2) return ((as64(m) >> idx) & 1ull) != 0ull;
  const unsigned bit = 1u << (idx & 31);
  const int wi = idx >> 5;
  unsigned hit = 0u;
#pragma unroll
  for (int k = 0; k < W; ++k) hit |= m[k] & (wi == k ? bit : 0u);
  return hit != 0u;
}
template <int W>
__device__ __forceinline__ void set_bit(unsigned (&m)[W], int idx) {
  if constexpr (W == 2) {
    const unsigned long long b = 1ull << idx;
    m[0] |= (unsigned)b;
    m[1] |= (unsigned)(b >> 32);
    return;
  }
  const unsigned bit = 1u << (idx & 31);
  const int wi = idx >> 5;
#pragma unroll
  for (int k = 0; k < W; ++k) m[k] |= (wi == k ? bit : 0u);
}
template <int W>
__device__ __forceinline__ void clear_bit(unsigned (&m)[W], int idx) {
  if constexpr (W == 2) {
    const unsigned long long b = 1ull << idx;
    m[0] &= ~(unsigned)b;
    m[1] &= ~(unsigned)(b >> 32);
    return;
  }
  const unsigned bit = 1u << (idx & 31);
  const int wi = idx >> 5;
#pragma unroll
  for (int k = 0; k < W; ++k) m[k] &= ~(wi == k ? bit : 0u);
}
template <int W>
__device__ __forceinline__ bool any_bit(const unsigned (&m)[W]) {
  unsigned o = 0;
#pragma unroll
  for (int k = 0; k < W; ++k) o |= m[k];
  return o != 0;
}
// lowest set bit of a mask, or -1
template <int W>
__device__ __forceinline__ int lowest_bit(const unsigned (&m)[W]) {
  int r = -1;
#pragma unroll
  for (int k = W - 1; k >= 0; --k)
    if (m[k]) r = k * 32 + __ffs(m[k]) - 1;
  return r;
}
// highest set bit of a mask, or -1
template <int W>
__device__ __forceinline__ int highest_bit(const unsigned (&m)[W]) {
  int r = -1;
#pragma unroll
  for (int k = 0; k < W; ++k)
    if (m[k]) r = k * 32 + 31 - __clz(m[k]);
  return r;
}
// word k of the set {t, t+1, ...}
__device__ __forceinline__ unsigned ge_word(int t, int k) {
  const int lo = k * 32;
  return t <= lo ? 0xffffffffu : (t >= lo + 32 ? 0u : (0xffffffffu << (t - lo)));
}
template <int C, typename T>
__device__ __forceinline__ T pick(const T (&a)[C], int s) {
  T v = a[0];
#pragma unroll
  for (int k = 1; k < C; ++k)
    if (s == k) v = a[k];
  return v;
}
template <int C, typename T>
__device__ __forceinline__ void put(T (&a)[C], int s, T v) {
#pragma unroll
  for (int k = 0; k < C; ++k)
    if (s == k) a[k] = v;
}

// one-hot word w of the set {idx}; empty for idx < 0
__device__ __forceinline__ unsigned onehot_word(int idx, int w) {
  return (idx >> 5) == w ? 1u << (idx & 31) : 0u;
}
// The one-hot mask of idx (empty for idx < 0) and the set {t, t+1, ...} as whole masks. With two
// words (33..64 rows, the headline size) a 64-bit shift does both words at once.
template <int W>
__device__ __forceinline__ void onehot_mask(int idx, unsigned (&m)[W]) {
  if constexpr (W == 2) {
    const unsigned long long b = idx >= 0 ? 1ull << idx : 0ull;
    m[0] = (unsigned)b;
    m[1] = (unsigned)(b >> 32);
  } else {
#pragma unroll
    for (int w = 0; w < W; ++w) m[w] = onehot_word(idx, w);
  }
}
template <int W>
__device__ __forceinline__ void ge_mask(int t, unsigned (&m)[W]) {
  if constexpr (W == 2) {
    const unsigned long long b = t >= 64 ? 0ull : (~0ull << (t > 0 ? t : 0));
    m[0] = (unsigned)b;
    m[1] = (unsigned)(b >> 32);
  } else {
#pragma unroll
    for (int w = 0; w < W; ++w) m[w] = ge_word(t, w);
  }
}

template <int W>
__device__ __forceinline__ bool intersects(const unsigned (&a)[W], const unsigned (&b)[W]) {
  unsigned o = 0u;
#pragma unroll
  for (int k = 0; k < W; ++k) o |= a[k] & b[k];
  return o != 0u;
}

// The matching as the lane sees it: mr[s] = row matched to the lane's column s (-1 = none).
// For up to 4 columns per lane the row is also kept as a one-hot mask, so that "is my row in
// this set" is two logic operations instead of a variable shift and select per word.
template <int CPL>
struct Match {
  static constexpr int W = CPL;
  static constexpr bool CACHED = CPL <= 4;
  int mr[CPL];
  unsigned oh[CACHED ? CPL : 1][CACHED ? CPL : 1];

  __device__ __forceinline__ void reset() {
#pragma unroll
    for (int s = 0; s < CPL; ++s) mr[s] = -1;
    if constexpr (CACHED) {
#pragma unroll
      for (int s = 0; s < CPL; ++s)
#pragma unroll
        for (int w = 0; w < W; ++w) oh[s][w] = 0u;
    }
  }
  __device__ __forceinline__ unsigned word(int s, int w) const {   // s, w compile-time after unrolling
    if constexpr (CACHED) return oh[s][w];
    else return onehot_word(mr[s], w);
  }
  // slot chosen at run time
  __device__ __forceinline__ void assign(int slot, int row) {
    unsigned rowmask[CPL];
    if constexpr (CACHED) onehot_mask<CPL>(row, rowmask);
#pragma unroll
    for (int s = 0; s < CPL; ++s) {
      const bool me = s == slot;
      mr[s] = me ? row : mr[s];
      if constexpr (CACHED) {
#pragma unroll
        for (int w = 0; w < W; ++w) oh[s][w] = me ? rowmask[w] : oh[s][w];
      }
    }
  }
  __device__ __forceinline__ int row_of(int slot) const { return pick<CPL>(mr, slot); }
  __device__ __forceinline__ bool in(const unsigned (&set)[CPL], int s) const {
    unsigned o = 0u;
#pragma unroll
    for (int w = 0; w < W; ++w) o |= set[w] & word(s, w);
    return o != 0u;
  }
  __device__ __forceinline__ void add_to(unsigned (&set)[CPL], int s) const {
#pragma unroll
    for (int w = 0; w < W; ++w) set[w] |= word(s, w);
  }
  // unmatch the columns whose row is in `rows`
  __device__ __forceinline__ void release(const unsigned (&rows)[CPL]) {
#pragma unroll
    for (int s = 0; s < CPL; ++s) {
      if (in(rows, s)) {
        mr[s] = -1;
        if constexpr (CACHED) {
#pragma unroll
          for (int w = 0; w < W; ++w) oh[s][w] = 0u;
        }
      }
    }
  }
};

// The lowest column, over the whole warp, whose slot qualifies (qualifies(s) is asked for every slot s of the
// lane), with the row matched to it (-1: the column is free), the lane that owns it and its slot there. Returns
// false when no column qualifies. With one or two columns per lane, column and row travel packed in one word
// through a single minimum over the warp (the column, in the upper half, decides); with more columns per lane
// packing every slot costs more than it saves, and the lowest proposing lane is found by a vote and read by
// shuffles. (Measured on the Birkhoff kernel, N = 64: 40.5 ms packed against 41.9 ms; N = 128: 278 ms packed
// against 265 ms.)
template <int CPL, class Q>
__device__ __forceinline__ bool lowest_qualifying_column(int lane, const Match<CPL>& M, Q qualifies, int& col,
                                                         int& row, int& owner_lane, int& slot) {
  if constexpr (CPL <= 2) {
    unsigned key = 0xffffffffu;
#pragma unroll
    for (int ss = 0; ss < CPL; ++ss) {
      const int s = CPL - 1 - ss;
      if (qualifies(s)) key = ((unsigned)(lane * CPL + s) << 16) | ((unsigned)M.mr[s] & 0xffffu);
    }
    key = __reduce_min_sync(FULL, key);
    if (key == 0xffffffffu) return false;
    col = (int)(key >> 16);
    const int r = (int)(key & 0xffffu);
    row = r == 0xffff ? -1 : r;
    owner_lane = col / CPL;
    slot = col % CPL;
    return true;
  } else {
    int ms = -1;
#pragma unroll
    for (int ss = 0; ss < CPL; ++ss) {
      const int s = CPL - 1 - ss;
      if (qualifies(s)) ms = s;
    }
    const unsigned ball = __ballot_sync(FULL, ms >= 0);
    if (ball == 0u) return false;
    owner_lane = __ffs(ball) - 1;
    slot = __shfl_sync(FULL, ms, owner_lane);
    col = owner_lane * CPL + slot;
    row = __shfl_sync(FULL, M.row_of(slot), owner_lane);
    return true;
  }
}

// Level of the search history (levels 1..level, W words each) that contains row r, 0 if none does. Every row
// belongs to one level only, so lane d can look at level d and a vote finds it.
template <int W>
__device__ __forceinline__ int level_of_row(const unsigned* hist, int level, int r, int lane) {
  int lvl = 0;
  for (int base = 1; base <= level && lvl == 0; base += 32) {
    const int d = base + lane;
    const bool at = d <= level && ((hist[d * W + (r >> 5)] >> (r & 31)) & 1u);
    const unsigned found = __ballot_sync(FULL, at);
    if (found != 0u) lvl = base + __ffs(found) - 1;
  }
  return lvl;
}

// ---- the matrix in shared memory --------------------------------------------------------
// Rows [0, split) live in this CTA's shared memory, rows [split, N) in the
// partner CTA of the cluster (far == generic pointer into its shared memory).
// Without a cluster split >= N and far is unused.
struct MatView {
  int* near_;
  int* far_;
  int S;      // row stride in ints, a multiple of CPL
  int split;  // first row held by the partner CTA
  __device__ __forceinline__ int* row(int r) const {
    return r < split ? near_ + r * S : far_ + (r - split) * S;
  }
};

template <int CPL>
struct RowVec {
  int v[CPL];
};

// Vector load of the lane's CPL consecutive columns of one row. The caller
// guarantees lane*CPL < S.
template <int CPL>
__device__ __forceinline__ RowVec<CPL> load_cols(const int* rowp, int lane) {
  RowVec<CPL> r;
  if constexpr (CPL == 1) {
    r.v[0] = rowp[lane];
  } else if constexpr (CPL == 2) {
    int2 t = *reinterpret_cast<const int2*>(rowp + lane * 2);
    r.v[0] = t.x; r.v[1] = t.y;
  } else if constexpr (CPL == 4) {
    int4 t = *reinterpret_cast<const int4*>(rowp + lane * 4);
    r.v[0] = t.x; r.v[1] = t.y; r.v[2] = t.z; r.v[3] = t.w;
  } else {
    int4 t = *reinterpret_cast<const int4*>(rowp + lane * 8);
    int4 q = *reinterpret_cast<const int4*>(rowp + lane * 8 + 4);
    r.v[0] = t.x; r.v[1] = t.y; r.v[2] = t.z; r.v[3] = t.w;
    r.v[4] = q.x; r.v[5] = q.y; r.v[6] = q.z; r.v[7] = q.w;
  }
  return r;
}

// The same matrix held as 16-bit entries (all values <= 65535): half the shared memory per
// matrix, hence twice the matrices per SM for the kernels that shared memory limits.
struct MatView16 {
  unsigned short* base;
  int S;   // row stride in entries, a multiple of CPL
  __device__ __forceinline__ unsigned short* row(int r) const { return base + r * S; }
};

template <int CPL>
__device__ __forceinline__ RowVec<CPL> load_cols(const unsigned short* rowp, int lane) {
  RowVec<CPL> r;
  if constexpr (CPL == 1) {
    r.v[0] = rowp[lane];
  } else if constexpr (CPL == 2) {
    const unsigned t = *reinterpret_cast<const unsigned*>(rowp + lane * 2);
    r.v[0] = t & 0xffffu; r.v[1] = t >> 16;
  } else if constexpr (CPL == 4) {
    const uint2 t = *reinterpret_cast<const uint2*>(rowp + lane * 4);
    r.v[0] = t.x & 0xffffu; r.v[1] = t.x >> 16; r.v[2] = t.y & 0xffffu; r.v[3] = t.y >> 16;
  } else {
    const uint4 t = *reinterpret_cast<const uint4*>(rowp + lane * 8);
    r.v[0] = t.x & 0xffffu; r.v[1] = t.x >> 16; r.v[2] = t.y & 0xffffu; r.v[3] = t.y >> 16;
    r.v[4] = t.z & 0xffffu; r.v[5] = t.z >> 16; r.v[6] = t.w & 0xffffu; r.v[7] = t.w >> 16;
  }
  return r;
}

// ---- bulk asynchronous copy global -> shared with an mbarrier ---------------------------

__device__ __forceinline__ unsigned smem_addr(const void* p) {
  return static_cast<unsigned>(__cvta_generic_to_shared(p));
}

// Issued by one lane. bytes is a multiple of 16, both addresses 16-byte aligned,
// bytes < 2^20 (transaction-count range of an mbarrier phase).
__device__ __forceinline__ void bulk_load_issue(void* smem_dst, const void* gmem_src, unsigned bytes,
                                                unsigned long long* mbar) {
  unsigned bar = smem_addr(mbar);
  asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_addr(smem_dst)),
      "l"(gmem_src), "r"(bytes), "r"(bar)
      : "memory");
}

// All lanes wait for phase 0 of the barrier. The wait is bounded: false means
// the copy did not land within the limit (never observed; reported, not spun on).
__device__ __forceinline__ bool bulk_load_wait(unsigned long long* mbar) {
  unsigned bar = smem_addr(mbar);
  for (int it = 0; it < (1 << 22); ++it) {
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar)
        : "memory");
    if (done) return true;
  }
  return false;
}

// The same barrier used for a SERIES of bulk copies into one staging buffer: initialised once, armed and
// waited for once per copy (the phase parity alternates), invalidated before its memory is used for
// anything else.
__device__ __forceinline__ void mbar_init(unsigned long long* mbar) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(mbar)));
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_inval(unsigned long long* mbar) {
  asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_addr(mbar)) : "memory");
}
// Issued by one thread. bytes is a multiple of 16, both addresses 16-byte aligned, bytes < 2^20.
__device__ __forceinline__ void mbar_bulk_copy(void* smem_dst, const void* gmem_src, unsigned bytes,
                                               unsigned long long* mbar) {
  const unsigned bar = smem_addr(mbar);
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_addr(smem_dst)),
      "l"(gmem_src), "r"(bytes), "r"(bar)
      : "memory");
}
// Bounded wait for the phase with the given parity; false if the copy did not land within the limit.
__device__ __forceinline__ bool mbar_wait(unsigned long long* mbar, unsigned parity) {
  const unsigned bar = smem_addr(mbar);
  for (int it = 0; it < (1 << 22); ++it) {
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}
// Rows per staged copy: as many whole rows of N int32 as fit `stage_bytes`, such that every copy is a
// multiple of 16 bytes; 0 when the matrix cannot be staged (odd N, misaligned source, no room for a row).
__device__ __forceinline__ int staged_rows(const int32_t* src, int N, size_t stage_bytes) {
  if ((N & 1) || (reinterpret_cast<uintptr_t>(src) & 15)) return 0;
  int rows = (int)(stage_bytes / ((size_t)N * 4));
  if (N & 3) rows &= ~1;   // N = 2 mod 4: an even number of rows makes a multiple of 16 bytes
  return rows;
}

// ---- cluster helpers ---------------------------------------------------------------------

__device__ __forceinline__ unsigned cluster_ctarank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// generic address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ int* map_to_cta(int* local_smem_ptr, unsigned rank) {
  unsigned long long out;
  asm volatile("mapa.u64 %0, %1, %2;" : "=l"(out) : "l"((unsigned long long)local_smem_ptr), "r"(rank));
  return reinterpret_cast<int*>(out);
}

// ---- load one matrix into shared memory (one warp) ----------------------------------------
// Copies rows [r0, r1) of the N x N matrix at g into dst with row stride S.
// Returns false if the bounded wait of the bulk copy ran out.
__device__ __forceinline__ bool load_rows(int* dst, const int32_t* g, int N, int S, int r0, int r1, int lane,
                                          unsigned long long* mbar) {
  const int rows = r1 - r0;
  if (rows <= 0) return true;
  const size_t bytes = (size_t)rows * N * 4;
  const int32_t* src = g + (size_t)r0 * N;
  const bool bulk = (S == N) && (bytes % 16 == 0) && ((reinterpret_cast<uintptr_t>(src) & 15) == 0) &&
                    bytes < (1u << 20);
  if (bulk) {
    if (lane == 0) bulk_load_issue(dst, src, (unsigned)bytes, mbar);
    __syncwarp();
    return bulk_load_wait(mbar);
  }
  for (int r = 0; r < rows; ++r)
    for (int c = lane; c < S; c += 32) dst[r * S + c] = c < N ? src[(size_t)r * N + c] : 0;
  __syncwarp();
  return true;
}

// ---- per-warp set-up shared by the kernels ----------------------------------------------------
// Shared memory of one warp: [matrix rows held here][hist: (N+1)*W words of search levels, then N*W
// words of per-row memo][x: N shorts][mbarrier][flag].
// In cluster mode the grid has two CTAs (one warp each) per matrix: CTA 0 of the pair
// works, CTA 1 loads rows [split, N) into its own shared memory and then only keeps
// them available to CTA 0 (distributed shared memory) until the final cluster barrier.
struct WarpCtx {
  int b;          // matrix index
  int lane;
  MatView M;
  unsigned* hist;
  short* x;
  bool loaded;    // the matrix arrived in shared memory
  bool worker;    // false: this warp has nothing more to do (return after cluster_epilogue)
};

__host__ __device__ inline size_t align16(size_t v) { return (v + 15) & ~(size_t)15; }
__host__ __device__ inline size_t hist_bytes_for(int N, int W) { return align16((size_t)(2 * N + 1) * W * 4); }
__host__ __device__ inline size_t warp_smem_bytes(int N, int S, int W, bool cluster) {
  const int rows_here = cluster ? (N + 1) / 2 : N;
  return align16((size_t)rows_here * S * 4) + hist_bytes_for(N, W) + align16((size_t)N * 2) + 16;
}

template <int CPL, bool CLUSTER>
__device__ __forceinline__ WarpCtx warp_prologue(int B, int N, int S, const int32_t* demand,
                                                 unsigned char* smem_raw) {
  WarpCtx cx;
  cx.lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int wpb = blockDim.x >> 5;
  const int split = CLUSTER ? (N + 1) / 2 : N;
  const int rows_here = CLUSTER ? split : N;
  const size_t mat_bytes = align16((size_t)rows_here * S * 4);
  const size_t hist_bytes = hist_bytes_for(N, CPL);
  const size_t x_bytes = align16((size_t)N * 2);
  unsigned char* base = smem_raw + (size_t)warp * warp_smem_bytes(N, S, CPL, CLUSTER);
  int* mat = reinterpret_cast<int*>(base);
  cx.hist = reinterpret_cast<unsigned*>(base + mat_bytes);
  cx.x = reinterpret_cast<short*>(base + mat_bytes + hist_bytes);
  unsigned long long* mbar = reinterpret_cast<unsigned long long*>(base + mat_bytes + hist_bytes + x_bytes);
  int* peer_flag = reinterpret_cast<int*>(mbar + 1);
  cx.M.near_ = mat;
  cx.M.far_ = mat;
  cx.M.S = S;
  cx.M.split = split;
  cx.worker = true;
  cx.loaded = true;
  if constexpr (CLUSTER) {
    const unsigned crank = cluster_ctarank();
    cx.b = blockIdx.x >> 1;   // grid = 2 B, so always < B
    const int32_t* g = demand + (size_t)cx.b * N * N;
    if (crank == 0) cx.loaded = load_rows(mat, g, N, S, 0, split, cx.lane, mbar);
    else cx.loaded = load_rows(mat, g, N, S, split, N, cx.lane, mbar);
    if (cx.lane == 0) *peer_flag = cx.loaded ? 1 : 0;
    cx.M.far_ = map_to_cta(mat, 1);
    cluster_sync_all();
    if (crank != 0) cx.worker = false;
    else cx.loaded = cx.loaded && (*map_to_cta(peer_flag, 1) != 0);
  } else {
    cx.b = blockIdx.x * wpb + warp;
    if (cx.b >= B) { cx.worker = false; return cx; }
    cx.loaded = load_rows(mat, demand + (size_t)cx.b * N * N, N, S, 0, N, cx.lane, mbar);
  }
  return cx;
}

// Variant with the working copy of the matrix in caller-provided global memory (row stride
// S ints, one N x S slab per matrix): shared memory then holds only hist and x, so many more
// warps fit on an SM. Suits kernels that touch the matrix a few times per matching.
__host__ __device__ inline size_t warp_smem_bytes_global(int N, int W) {
  return hist_bytes_for(N, W) + align16((size_t)N * 2);
}

template <int CPL>
__device__ __forceinline__ WarpCtx warp_prologue_global(int B, int N, int S, const int32_t* demand,
                                                        int32_t* scratch, unsigned char* smem_raw) {
  WarpCtx cx;
  cx.lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int wpb = blockDim.x >> 5;
  unsigned char* base = smem_raw + (size_t)warp * warp_smem_bytes_global(N, CPL);
  cx.hist = reinterpret_cast<unsigned*>(base);
  cx.x = reinterpret_cast<short*>(base + hist_bytes_for(N, CPL));
  cx.b = blockIdx.x * wpb + warp;
  cx.worker = cx.b < B;
  cx.loaded = true;
  cx.M.S = S;
  cx.M.split = N;
  cx.M.near_ = cx.M.far_ = nullptr;
  if (!cx.worker) return cx;
  int* mat = scratch + (size_t)cx.b * N * S;
  cx.M.near_ = cx.M.far_ = mat;
  const int32_t* src = demand + (size_t)cx.b * N * N;
  for (int r = 0; r < N; ++r)
    for (int c = cx.lane; c < S; c += 32) mat[(size_t)r * S + c] = c < N ? src[(size_t)r * N + c] : 0;
  __syncwarp();
  return cx;
}

// One warp: rows of N int32 arrive in `stage` by bulk copies of rows_per_copy rows each and are narrowed to
// 16 bits into dst (row stride S, padding columns zeroed). Kept out of line so that its registers do not
// count against the kernel that calls it once. Returns false if a copy did not land within its bounded wait.
static __device__ __noinline__ bool stage_and_narrow(const int32_t* src, int N, int S, int rows_per_copy, int lane,
                                              unsigned short* dst, int* stage, unsigned long long* mbar) {
  if (lane == 0) mbar_init(mbar);
  __syncwarp();
  unsigned parity = 0;
  bool ok = true;
  for (int r0 = 0; r0 < N; r0 += rows_per_copy) {
    const int rows = min(rows_per_copy, N - r0);
    if (lane == 0) mbar_bulk_copy(stage, src + (size_t)r0 * N, (unsigned)(rows * N * 4), mbar);
    __syncwarp();
    if (!mbar_wait(mbar, parity)) {
      mbar_wait(mbar, parity);   // one more bounded wait for the copy in flight before giving up
      ok = false;
      break;
    }
    parity ^= 1u;
    for (int r = 0; r < rows; ++r)
      for (int c = lane; c < S; c += 32)
        dst[(r0 + r) * S + c] = c < N ? (unsigned short)stage[r * N + c] : (unsigned short)0;
    __syncwarp();   // the staging rows are free again
  }
  if (ok && lane == 0) mbar_inval(mbar);
  __syncwarp();
  return ok;
}

// Variant for matrices whose entries all fit 16 bits: the warp's shared memory is
// [N x S entries of 16 bits][hist][x]; the entries are narrowed while they are loaded.
__host__ __device__ inline size_t warp_smem_bytes16(int N, int S, int W) {
  return align16((size_t)N * S * 2) + hist_bytes_for(N, W) + align16((size_t)N * 2);
}

struct WarpCtx16 {
  int b;
  int lane;
  MatView16 M;
  unsigned* hist;
  short* x;
  bool worker;
  bool loaded;    // false: a bulk copy did not land within its bounded wait
};

// STAGED: the rows come in by bulk asynchronous copies and are narrowed from a staging area (scoring, whose
// short launches are dominated by the load); otherwise plain coalesced loads narrow on the fly (greedy: with
// the staged loop in its prologue the compiler gives the whole kernel 128 registers instead of 64, 16
// instead of 22 warps per SM, measured 12.4 ms against 12.1 ms on 4096 matrices of 64 ranks).
template <int CPL, bool STAGED>
__device__ __forceinline__ WarpCtx16 warp_prologue16(int B, int N, int S, const int32_t* demand,
                                                     unsigned char* smem_raw) {
  WarpCtx16 cx;
  cx.lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int wpb = blockDim.x >> 5;
  unsigned char* base = smem_raw + (size_t)warp * warp_smem_bytes16(N, S, CPL);
  const size_t mat_bytes = align16((size_t)N * S * 2);
  cx.M.base = reinterpret_cast<unsigned short*>(base);
  cx.M.S = S;
  cx.hist = reinterpret_cast<unsigned*>(base + mat_bytes);
  cx.x = reinterpret_cast<short*>(base + mat_bytes + hist_bytes_for(N, CPL));
  cx.b = blockIdx.x * wpb + warp;
  cx.worker = cx.b < B;
  cx.loaded = true;
  if (!cx.worker) return cx;
  const int32_t* src = demand + (size_t)cx.b * N * N;
  // The int32 rows come in by bulk asynchronous copies, a few rows at a time, into the memory that will
  // hold the search history later (nothing lives there yet), and are narrowed from there; the barrier of
  // the copies borrows the first bytes of x. Matrices that cannot be staged take plain loads.
  const int rows_per_copy = STAGED ? staged_rows(src, N, hist_bytes_for(N, CPL)) : 0;
  if (STAGED && rows_per_copy > 0) {
    cx.loaded = stage_and_narrow(src, N, S, rows_per_copy, cx.lane, cx.M.base, reinterpret_cast<int*>(cx.hist),
                                 reinterpret_cast<unsigned long long*>(cx.x));
    return cx;
  }
  for (int r = 0; r < N; ++r)
    for (int c = cx.lane; c < S; c += 32)
      cx.M.base[r * S + c] = c < N ? (unsigned short)src[(size_t)r * N + c] : (unsigned short)0;
  __syncwarp();
  return cx;
}

// Every warp of a cluster launch passes here exactly once before it returns.
template <bool CLUSTER>
__device__ __forceinline__ void cluster_epilogue() {
  if constexpr (CLUSTER) cluster_sync_all();
}

// ---- lexicographically smallest perfect matching -------------------------------------------
//
// State: C[s] = set of rows adjacent to the lane's column s in the graph (tight
// edges for the greedy step, positive entries for Birkhoff), mr[s] = row matched
// to that column, x[r] = column matched to row r (shared memory, one entry per
// row). On entry (mr, x) is some perfect matching of the graph. For each row i
// in order the routine finds the lowest column that row i can take in a perfect
// matching that keeps rows < i fixed: an edge (i, j) outside the matching is
// usable iff row mr[j] reaches row i along alternating steps r -> r' (r adjacent
// to the column of r') among the rows not yet fixed; the matching is then rotated
// along that cycle. hist holds one row set per search level to retrace the cycle.
//
// Only the window [start, last] of rows is visited. The caller guarantees that the
// matching already equals the answer on rows < start, and that every row > last
// was settled by an earlier call, with no row >= it re-matched and no edge added
// since: its search could only find less now, so its column stands. A rotation at
// row i moves rows above i and widens the window accordingly.
// Rows i that have, below their own column, a column they are adjacent to whose row lies
// above i: only those can move to a lower column. Uniform result. With gt(c) = rows matched
// to a column > c (a suffix OR over the lanes), row i qualifies through column c iff
// i is adjacent to c, i < mr[c] and i is in gt(c).
template <int CPL>
__device__ __forceinline__ void candidate_rows(int lane, const unsigned (&C)[CPL][CPL], const Match<CPL>& M,
                                               unsigned (&cand)[CPL]) {
  constexpr int W = CPL;
  unsigned own[W];
#pragma unroll
  for (int w = 0; w < W; ++w) own[w] = 0u;
#pragma unroll
  for (int s = 0; s < CPL; ++s) M.add_to(own, s);
  unsigned above[W];   // rows matched to the columns of higher lanes
#pragma unroll
  for (int w = 0; w < W; ++w) {
    unsigned v = own[w];
#pragma unroll
    // (a lane whose source would lie beyond lane 31 gets its own value back: harmless in an OR)
    for (int o = 1; o < 32; o <<= 1) v |= __shfl_down_sync(FULL, v, o);
    // v now covers this lane and all higher ones; every row is matched to one column only, so
    // taking the lane's own rows out leaves exactly the rows of the higher lanes
    above[w] = v & ~own[w];
  }
  // A row can only move if some row above it is adjacent to its own column (the last step of the
  // alternating cycle back into it): rows without such a neighbour are dropped here, which spares
  // them a search that would reach nobody.
  unsigned acc[W], entered[W];
#pragma unroll
  for (int w = 0; w < W; ++w) acc[w] = entered[w] = 0u;
#pragma unroll
  for (int ss = 0; ss < CPL; ++ss) {
    const int s = CPL - 1 - ss;   // from the lane's highest column down, growing gt as we go
    if (M.mr[s] >= 0) {
      unsigned higher = 0u, gem[W];
      ge_mask<W>(M.mr[s], gem);
#pragma unroll
      for (int w = 0; w < W; ++w) {
        const unsigned ge = gem[w];
        acc[w] |= C[s][w] & above[w] & ~ge;
        higher |= C[s][w] & ge & ~M.word(s, w);
      }
      if (higher != 0u) {
#pragma unroll
        for (int w = 0; w < W; ++w) entered[w] |= M.word(s, w);
      }
    }
    M.add_to(above, s);
  }
#pragma unroll
  for (int w = 0; w < W; ++w) cand[w] = __reduce_or_sync(FULL, acc[w]) & __reduce_or_sync(FULL, entered[w]);
}

// Memo carried from one call to the next when the graph only loses edges between calls
// (Birkhoff): known = rows whose last search found no lower column and whose searched set
// (the rows that could reach them) is recorded; desc[r] (shared memory, W words per row,
// after the level history) = rows that have r in their recorded set. Such a row needs no new
// search until a row of its recorded set changes column: new alternating steps only lead
// INTO rows that changed, so a row that reaches it through them would have to pass a changed
// row that already reached it before. changed = rows whose column changed since the last call.
template <int W>
struct CanonMemo {
  // Up to 128 rows the per-row records live in registers: the lane keeps desc of rows
  // lane, lane+32, ... (word k of a row set, bit `lane`), so collecting and recording are a
  // few logic operations and one OR-reduction per word. Above that they live in shared memory.
  static constexpr bool IN_REGS = W <= 4;
  unsigned known[W];
  unsigned changed[W];
  unsigned dreg[IN_REGS ? W : 1][IN_REGS ? W : 1];
  __device__ __forceinline__ void reset() {
#pragma unroll
    for (int w = 0; w < W; ++w) known[w] = changed[w] = 0u;
    if constexpr (IN_REGS) {
#pragma unroll
      for (int k = 0; k < W; ++k)
#pragma unroll
        for (int w = 0; w < W; ++w) dreg[k][w] = 0u;
    }
  }
};

// rows recorded as depending on any row of `rows` are added to out; their entries are consumed
template <int W>
__device__ __forceinline__ void collect_dependants(int N, int lane, const unsigned (&rows)[W], unsigned* desc,
                                                   CanonMemo<W>& memo, unsigned (&out)[W]) {
  if constexpr (CanonMemo<W>::IN_REGS) {
    unsigned acc[W];
#pragma unroll
    for (int w = 0; w < W; ++w) acc[w] = 0u;
#pragma unroll
    for (int k = 0; k < W; ++k) {
      if ((rows[k] >> lane) & 1u) {
#pragma unroll
        for (int w = 0; w < W; ++w) { acc[w] |= memo.dreg[k][w]; memo.dreg[k][w] = 0u; }
      }
    }
#pragma unroll
    for (int w = 0; w < W; ++w) out[w] |= __reduce_or_sync(FULL, acc[w]);
  } else {
    unsigned left[W];
#pragma unroll
    for (int w = 0; w < W; ++w) left[w] = rows[w];
    for (int it = 0; it < N; ++it) {
      const int r = lowest_bit<W>(left);
      if (r < 0) break;
      clear_bit<W>(left, r);
#pragma unroll
      for (int w = 0; w < W; ++w) out[w] |= desc[MS_AT(r, N) * W + w];
    }
    __syncwarp();
    // lane l clears the entries of the rows l, l+32, ... that were just read
#pragma unroll
    for (int k = 0; k < W; ++k) {
      if ((rows[k] >> lane) & 1u) {
#pragma unroll
        for (int w = 0; w < W; ++w) desc[MS_AT(k * 32 + lane, N) * W + w] = 0u;
      }
    }
    __syncwarp();
  }
}

// record that row i (one-hot imask) was searched and depends on the rows of anc
template <int W>
__device__ __forceinline__ void record_search(int lane, int i, const unsigned (&imask)[W], const unsigned (&anc)[W],
                                              unsigned* desc, CanonMemo<W>& memo) {
#pragma unroll
  for (int k = 0; k < W; ++k) {
    if ((anc[k] >> lane) & 1u) {
      if constexpr (CanonMemo<W>::IN_REGS) {
#pragma unroll
        for (int w = 0; w < W; ++w) memo.dreg[k][w] |= imask[w];
      } else {
        desc[(k * 32 + lane) * W + (i >> 5)] |= 1u << (i & 31);
      }
    }
    memo.known[k] |= imask[k];
  }
  if constexpr (!CanonMemo<W>::IN_REGS) __syncwarp();
}

// One row set of the search history (W words at hist + level * W). The set is uniform and EVERY lane stores
// it (same address, same value: one shared-memory transaction), so that a lane which reads the history later
// reads what it wrote itself, in program order: no warp barrier is needed between the store and the loads. The
// matching x[] is kept the same way (every lane makes every update). Two words go in one 8-byte store, four
// or eight in 16-byte stores (hist is 16-byte aligned and W * 4 divides 16 or is a multiple of it).
template <int W>
__device__ __forceinline__ void hist_store(unsigned* hist, int level, const unsigned (&F)[W], int /*lane*/) {
  if constexpr (W == 2) {
    *reinterpret_cast<uint2*>(hist + level * 2) = make_uint2(F[0], F[1]);
  } else if constexpr (W % 4 == 0) {
#pragma unroll
    for (int q = 0; q < W; q += 4)
      *reinterpret_cast<uint4*>(hist + level * W + q) = make_uint4(F[q], F[q + 1], F[q + 2], F[q + 3]);
  } else {
#pragma unroll
    for (int w = 0; w < W; ++w) hist[level * W + w] = F[w];
  }
}
template <int W>
__device__ __forceinline__ void hist_load(const unsigned* hist, int level, unsigned (&H)[W]) {
  if constexpr (W == 2) {
    const uint2 v = *reinterpret_cast<const uint2*>(hist + level * 2);
    H[0] = v.x;
    H[1] = v.y;
  } else {
#pragma unroll
    for (int w = 0; w < W; ++w) H[w] = hist[level * W + w];
  }
}

template <int CPL, bool MEMO>
__device__ __forceinline__ bool canonicalise(int N, int lane, int start, int last,
                                             const unsigned (&C)[CPL][CPL], Match<CPL>& M, short* x,
                                             unsigned* hist, CanonMemo<CPL>& memo,
                                             unsigned (&work)[MOESCHED_WORK_FIELDS]) {
  constexpr int W = CPL;
  unsigned* desc = hist + (N + 1) * W;
  bool ok_all = true;
  unsigned cand[W], stale[W];   // stale: rows whose recorded set contains a changed row
#pragma unroll
  for (int w = 0; w < W; ++w) stale[w] = 0u;
  if constexpr (MEMO) {
    collect_dependants<W>(N, lane, memo.changed, desc, memo, stale);
#pragma unroll
    for (int w = 0; w < W; ++w) {
      stale[w] |= memo.changed[w];
      memo.known[w] &= ~stale[w];    // rows before `start` keep their column but lose their record
      memo.changed[w] = 0u;
    }
  }
  candidate_rows<CPL>(lane, C, M, cand);
  // rows still to be looked at: those that could move, from `start` up to the last changed row,
  // not covered by a record that still holds. Rebuilt only after a rotation; otherwise the row just
  // searched is simply struck off.
  unsigned todo[W];
  {
    unsigned lo[W], hi[W];
    ge_mask<W>(start, lo);
    ge_mask<W>(last + 1, hi);
#pragma unroll
    for (int w = 0; w < W; ++w) {
      unsigned need = cand[w] & lo[w] & ~hi[w];
      if constexpr (MEMO) need &= ~memo.known[w];
      todo[w] = need;
    }
  }
  for (int guard = 0; guard < N; ++guard) {
    const int i = lowest_bit<W>(todo);
    if (i < 0) break;
    const int xi = x[MS_AT(i, N)];
    work[WK_SWEEP]++;
    // backward search from row i among the rows >= i; the one-hot mask of i and the set {i, i+1, ...}
    // come from isolating the lowest bit of todo
    unsigned anc[W], F[W], alive[W], imask[W];
    {
      bool below = true;   // all lower words of todo are empty
#pragma unroll
      for (int w = 0; w < W; ++w) {
        const unsigned lowbit = todo[w] & (0u - todo[w]);
        const bool here = below && todo[w] != 0u;
        imask[w] = here ? lowbit : 0u;
        alive[w] = here ? (0u - lowbit) & ~lowbit : (below ? 0u : 0xffffffffu);   // rows above i
        below = below && todo[w] == 0u;
        todo[w] &= ~imask[w];
        anc[w] = F[w] = imask[w];
      }
    }
    int level = 0;
    work[WK_POP]++;   // row i itself
    hist_store<W>(hist, 0, F, lane);
    // The lowest column below its own that row i is adjacent to and whose row lies above i: no lower column can
    // be had, so the search stops as soon as that row is reached (the levels up to there are those of the full
    // search, hence the same rotation). Used where it was measured to pay: in the Birkhoff steps (most
    // searches there end in a rotation) with one or two columns per lane (N = 64: 38.6 -> 37.4 ms; at N = 128,
    // and in the greedy steps, where most searches find nothing, finding the target costs more than it saves).
    constexpr bool EARLY = MEMO && CPL <= 2;
    int jstar = -1, cur = -1, L = 0, sl = 0;   // the column, the row that gives it up, its lane and slot
    unsigned target[W];
#pragma unroll
    for (int w = 0; w < W; ++w) target[w] = 0u;
    if constexpr (EARLY) {
      if (lowest_qualifying_column<CPL>(
              lane, M, [&](int s) { return lane * CPL + s < xi && M.mr[s] > i && intersects<W>(C[s], imask); },
              jstar, cur, L, sl))
        onehot_mask<W>(cur, target);
    }
    int early = 0;   // level at which the target row was reached
    for (int it = 0; it < N; ++it) {
      unsigned acc[W];
#pragma unroll
      for (int w = 0; w < W; ++w) acc[w] = 0u;
#pragma unroll
      for (int s = 0; s < CPL; ++s) {
        if (M.in(F, s)) {
#pragma unroll
          for (int w = 0; w < W; ++w) acc[w] |= C[s][w];
        }
      }
      bool grew = false;
#pragma unroll
      for (int w = 0; w < W; ++w) {
        const unsigned a = __reduce_or_sync(FULL, acc[w]) & alive[w];   // alive: rows >= i not reached yet
        alive[w] &= ~a;
        anc[w] |= a;
        F[w] = a;
        grew |= a != 0u;
      }
      work[WK_LEVEL]++;
      if (!grew) break;
      ++level;
#pragma unroll
      for (int w = 0; w < W; ++w) work[WK_POP] += __popc(F[w]);
      if constexpr (EARLY) {
        if (intersects<W>(F, target)) { early = level; break; }
      }
      hist_store<W>(hist, level, F, lane);
    }
    // otherwise: the lowest column row i may take (its own column always qualifies)
    if (early == 0 &&
        !lowest_qualifying_column<CPL>(
            lane, M, [&](int s) { return intersects<W>(C[s], imask) && M.in(anc, s); }, jstar, cur, L, sl)) {
      ok_all = false;
      continue;
    }
    if (jstar == xi) {
      // record: row i stays put until one of the rows that can reach it changes column
      if constexpr (MEMO) record_search<W>(lane, i, imask, anc, desc, memo);
    } else {
      // level at which that row was reached
      int lvl = early > 0 ? early : level_of_row<W>(hist, level, MS_AT(cur, N), lane);
      if (lvl == 0) ok_all = false;
      unsigned moved[W];
#pragma unroll
      for (int w = 0; w < W; ++w) moved[w] = imask[w];
      // walk towards row i: each row takes the column of its successor on the cycle
      while (lvl > 0) {
        unsigned Hm[W], cmask[W];
        onehot_mask<W>(cur, cmask);
        hist_load<W>(hist, lvl - 1, Hm);
#pragma unroll
        for (int w = 0; w < W; ++w) moved[w] |= cmask[w];
        int c2, nxt, L2, s2;
        if (!lowest_qualifying_column<CPL>(
                lane, M, [&](int s) { return M.in(Hm, s) && intersects<W>(C[s], cmask); }, c2, nxt, L2, s2)) {
          ok_all = false;
          break;
        }
        if (lane == L2) M.assign(s2, cur);
        x[MS_AT(cur, N)] = (short)c2;   // every lane (see hist_store)
        last = max(last, cur);
        cur = nxt;
        --lvl;
        work[WK_ROT]++;
      }
      if (lane == L) M.assign(sl, i);
      x[MS_AT(i, N)] = (short)jstar;
      if constexpr (MEMO) {
        // the moved rows changed column: every record that contains one of them is void
        unsigned hit[W];
#pragma unroll
        for (int w = 0; w < W; ++w) hit[w] = moved[w];
        collect_dependants<W>(N, lane, moved, desc, memo, hit);
#pragma unroll
        for (int w = 0; w < W; ++w) memo.known[w] &= ~hit[w];
      }
      candidate_rows<CPL>(lane, C, M, cand);
      unsigned lo[W], hi[W];
      ge_mask<W>(i + 1, lo);
      ge_mask<W>(last + 1, hi);
#pragma unroll
      for (int w = 0; w < W; ++w) {
        unsigned need = cand[w] & lo[w] & ~hi[w];
        if constexpr (MEMO) need &= ~memo.known[w];
        todo[w] = need;
      }
    }
  }
  return ok_all;
}

// ---- augmenting search on a 0/1 graph --------------------------------------------------------
// Augmenting search from free row f over alternating paths of the graph C (the support graph of
// the Birkhoff step, the tight edges of a greedy step).
// Among all augmenting paths it takes one whose lowest row is as high as possible: the
// search first uses only rows >= t = f and lowers t to the highest waiting row only when
// it is stuck, so the rows below the returned path keep their columns. [lo, hi] is widened
// to cover every row whose column changed. Returns false when no augmenting path exists
// (cannot happen for a balanced matrix).
template <int CPL>
__device__ __forceinline__ bool augment_from(int N, int lane, int f, const unsigned (&C)[CPL][CPL], Match<CPL>& M,
                                             short* x, int& lo, int& hi, unsigned (&changed)[CPL],
                                             unsigned (&work)[MOESCHED_WORK_FIELDS]) {
  constexpr int W = CPL;
  unsigned F[W], P[W];   // frontier rows; rows met but still below the threshold
#pragma unroll
  for (int w = 0; w < W; ++w) F[w] = P[w] = 0u;
  set_bit<W>(F, f);
  int t = f;
  unsigned at_or_above[W];   // rows >= t
  ge_mask<W>(t, at_or_above);
  unsigned visited = 0u;
  int par[CPL];
#pragma unroll
  for (int s = 0; s < CPL; ++s) par[s] = -1;
  int jf = -1;
  for (int it = 0; it < 2 * N + 2; ++it) {
    unsigned met[W];
#pragma unroll
    for (int w = 0; w < W; ++w) met[w] = 0u;
    int freeslot = -1;
#pragma unroll
    for (int ss = 0; ss < CPL; ++ss) {
      const int s = CPL - 1 - ss;
      if (!((visited >> s) & 1u)) {
        unsigned hit[W];
#pragma unroll
        for (int w = 0; w < W; ++w) hit[w] = C[s][w] & F[w];
        if (any_bit<W>(hit)) {
          visited |= 1u << s;
          par[s] = lowest_bit<W>(hit);
          if (M.mr[s] < 0) freeslot = s;
          else M.add_to(met, s);
        }
      }
    }
    work[WK_SCAN]++;
    const unsigned fb = __ballot_sync(FULL, freeslot >= 0);
    if (fb) {
      const int L = __ffs(fb) - 1;
      jf = L * CPL + __shfl_sync(FULL, freeslot, L);
      break;
    }
    bool grew = false;
#pragma unroll
    for (int w = 0; w < W; ++w) {
      const unsigned m = __reduce_or_sync(FULL, met[w]);
      const unsigned ge = at_or_above[w];
      F[w] = m & ge;
      P[w] |= m & ~ge;
      grew |= F[w] != 0u;
    }
    if (!grew) {
      const int r = highest_bit<W>(P);   // admit the highest waiting row, and only that one
      if (r < 0) return false;
      t = r;
      ge_mask<W>(t, at_or_above);
      clear_bit<W>(P, r);
      set_bit<W>(F, r);
    }
  }
  if (jf < 0) return false;
  int j = jf;
  for (int it = 0; it <= N; ++it) {
    const int L = j / CPL, sl = j % CPL;
    const int i = __shfl_sync(FULL, pick<CPL>(par, sl), L);
    const int jprev = x[MS_AT(i, N)];
    if (lane == L) M.assign(sl, i);
    x[MS_AT(i, N)] = (short)j;   // every lane (see hist_store)
    lo = min(lo, i);
    hi = max(hi, i);
    set_bit<W>(changed, i);
    work[WK_AUG]++;
    if (i == f) return true;
    j = jprev;
    if (j < 0) return false;
  }
  return false;
}

// ---- repair of a matching that lost an edge, canonical for the row that lost it -------------------------
// Birkhoff step: the entry (r0, c0) of a lexicographically smallest perfect matching has just vanished, so
// row r0 and column c0 are free. Rows below r0 keep their columns (they did so with more edges available).
// The columns that CAN be handed to r0 without touching rows below it are found by one forward search from
// the free column(s) over the rows above r0: a row adjacent to a column of the previous level could move
// there and release its own column. r0 takes the lowest such column it is adjacent to -- which is its column
// in the lexicographically smallest matching of the new graph -- and the rows on the way each move one step
// towards a free column. (When several entries vanished at once the free rows are handled lowest first; a
// free row above r0 releases nothing and is simply passed over. Each row's choice is the lowest among the
// matchings that leave the other free rows out, hence also among the complete ones if the rest can still be
// matched above it; if not, the caller's general search lowers the window as far as it has to.) This replaces an arbitrary augmenting path followed by a search (and
// usually a rotation) for row r0. Returns 1 when done (hi = highest row moved, `changed` gets the moved rows),
// 0 when r0 cannot be re-matched this way (the caller falls back to augment_from), -1 if an iteration limit
// was hit.
// With `may_lower` (the caller passes it when r0 is the only free row) the search does not give up when r0 is
// adjacent to no column that the rows above it can release: it admits the highest row BELOW r0 that is adjacent
// to a releasable column, continues from that row's column, and repeats until r0 can be served. The path then
// disturbs as few low rows as possible (as augment_from's does); r0's column is no longer final, `lo` is lowered
// to the lowest row that moved, and 2 is returned.
template <int CPL>
__device__ __forceinline__ int canonical_repair(int N, int lane, int r0, const unsigned (&C)[CPL][CPL], Match<CPL>& M,
                                                short* x, unsigned* hist, int& hi, unsigned (&changed)[CPL],
                                                unsigned (&work)[MOESCHED_WORK_FIELDS], bool may_lower, int& lo) {
  constexpr int W = CPL;
  unsigned alive[W], r0mask[W];
  ge_mask<W>(r0 + 1, alive);        // rows above r0 not reached yet
  onehot_mask<W>(r0, r0mask);
  unsigned front = 0u;              // bit s: the lane's column s belongs to the current level
#pragma unroll
  for (int s = 0; s < CPL; ++s)
    if (lane * CPL + s < N && M.mr[s] < 0) front |= 1u << s;
  if (__ballot_sync(FULL, front != 0u) == 0u) return 0;   // no free column: nothing to hand out
  unsigned freeable = front;        // bit s: column s is free or can be released
  int level = 0;
  bool lowered = false;
  unsigned below[W];                // rows below r0 not admitted yet
  {
    unsigned from_r0[W];
    ge_mask<W>(r0, from_r0);
#pragma unroll
    for (int w = 0; w < W; ++w) below[w] = ~from_r0[w];
  }
  int c0 = -1, cur = -1, L = 0, sl = 0;   // r0's column, the row that gives it up, its lane and slot
  // The lowest column r0 is adjacent to that is free or whose row lies above r0: if that row is reached, r0 can
  // have nothing lower and the search stops there (with one or two columns per lane, where finding it pays).
  constexpr bool EARLY = CPL <= 2;
  unsigned target[W];
#pragma unroll
  for (int w = 0; w < W; ++w) target[w] = 0u;
  int early = 0;
  int tc = -1, trow = -1, tL = 0, tsl = 0;   // that column, its row, lane and slot
  if constexpr (EARLY) {
    if (lowest_qualifying_column<CPL>(
            lane, M,
            [&](int s) { return lane * CPL + s < N && (M.mr[s] < 0 || M.mr[s] > r0) && intersects<W>(C[s], r0mask); },
            tc, trow, tL, tsl)) {
      if (trow >= 0) onehot_mask<W>(trow, target);
      else early = -1;   // the free column itself: nothing to search
    }
  }
  for (int round = 0; round <= N && early == 0; ++round) {
    for (int it = 0; it < N; ++it) {
      unsigned acc[W];
#pragma unroll
      for (int w = 0; w < W; ++w) acc[w] = 0u;
#pragma unroll
      for (int s = 0; s < CPL; ++s) {
        if ((front >> s) & 1u) {
#pragma unroll
          for (int w = 0; w < W; ++w) acc[w] |= C[s][w];
        }
      }
      unsigned nw[W];
      bool grew = false;
#pragma unroll
      for (int w = 0; w < W; ++w) {
        nw[w] = __reduce_or_sync(FULL, acc[w]) & alive[w];
        alive[w] &= ~nw[w];
        grew |= nw[w] != 0u;
      }
      work[WK_SCAN]++;
      if (!grew) break;
      ++level;
      if constexpr (EARLY) {
        if (intersects<W>(nw, target)) { early = level; break; }
      }
      hist_store<W>(hist, level, nw, lane);
      front = 0u;
#pragma unroll
      for (int s = 0; s < CPL; ++s)
        if (M.mr[s] >= 0 && M.in(nw, s)) front |= 1u << s;
      freeable |= front;
    }
    if (early != 0) break;
    // otherwise the lowest column that r0 is adjacent to and that can be released
    if (lowest_qualifying_column<CPL>(
            lane, M, [&](int s) { return ((freeable >> s) & 1u) && intersects<W>(C[s], r0mask); }, c0, cur, L, sl))
      break;
    c0 = -1;
    if (!may_lower) return 0;
    // admit the highest row below r0 that could move to a releasable column
    unsigned acc[W];
#pragma unroll
    for (int w = 0; w < W; ++w) acc[w] = 0u;
#pragma unroll
    for (int s = 0; s < CPL; ++s) {
      if ((freeable >> s) & 1u) {
#pragma unroll
        for (int w = 0; w < W; ++w) acc[w] |= C[s][w];
      }
    }
    unsigned waiting[W];
#pragma unroll
    for (int w = 0; w < W; ++w) waiting[w] = __reduce_or_sync(FULL, acc[w]) & below[w];
    const int t = highest_bit<W>(waiting);
    if (t < 0) return 0;
    clear_bit<W>(below, t);
    lowered = true;
    unsigned tmask[W];
    onehot_mask<W>(t, tmask);
    ++level;
    hist_store<W>(hist, level, tmask, lane);
    front = 0u;
#pragma unroll
    for (int s = 0; s < CPL; ++s)
      if (M.mr[s] >= 0 && M.in(tmask, s)) front |= 1u << s;
    freeable |= front;
    work[WK_SCAN]++;
  }
  if (early != 0) { c0 = tc; cur = trow; L = tL; sl = tsl; }
  if (c0 < 0) return -1;
  if (lane == L) M.assign(sl, r0);
  x[MS_AT(r0, N)] = (short)c0;   // every lane (see hist_store)
  set_bit<W>(changed, r0);
  hi = max(hi, r0);
  if (cur < 0) return 1;   // r0 took the free column itself
  int lvl = early > 0 ? early : level_of_row<W>(hist, level, MS_AT(cur, N), lane);
  if (lvl == 0) return -1;
  if (lowered) {
    // An admitted row joined through a column of ANY earlier level, so a row moves to the lowest column it is
    // adjacent to whose row was reached at an earlier level (or that is free); the levels still fall strictly.
    lo = min(lo, r0);
    for (int it = 0; it <= N; ++it) {
      unsigned cmask[W], Hm[W];
      onehot_mask<W>(cur, cmask);
#pragma unroll
      for (int w = 0; w < W; ++w) Hm[w] = 0u;
      for (int d = 1; d < lvl; ++d) {
        unsigned Hd[W];
        hist_load<W>(hist, d, Hd);
#pragma unroll
        for (int w = 0; w < W; ++w) Hm[w] |= Hd[w];
      }
      int c2, nxt, L2, s2;
      if (!lowest_qualifying_column<CPL>(
              lane, M,
              [&](int s) {
                return lane * CPL + s < N && (M.mr[s] < 0 || M.in(Hm, s)) && intersects<W>(C[s], cmask);
              },
              c2, nxt, L2, s2))
        return -1;
      if (lane == L2) M.assign(s2, cur);
      x[MS_AT(cur, N)] = (short)c2;
      set_bit<W>(changed, cur);
      hi = max(hi, cur);
      lo = min(lo, cur);
      work[WK_AUG]++;
      if (nxt < 0) return 2;   // took the free column
      cur = nxt;
      lvl = level_of_row<W>(hist, level, MS_AT(cur, N), lane);
      if (lvl == 0) return -1;
    }
    return -1;
  }
  for (int it = 0; it <= N; ++it) {
    // cur, reached at level lvl, moves to a column of level lvl - 1 (level 0: the free column)
    unsigned cmask[W];
    onehot_mask<W>(cur, cmask);
    int c2, nxt, L2, s2;
    bool found;
    if (lvl == 1) {
      found = lowest_qualifying_column<CPL>(
          lane, M, [&](int s) { return lane * CPL + s < N && M.mr[s] < 0 && intersects<W>(C[s], cmask); }, c2, nxt,
          L2, s2);
    } else {
      unsigned Hm[W];
      hist_load<W>(hist, lvl - 1, Hm);
      found = lowest_qualifying_column<CPL>(
          lane, M, [&](int s) { return M.in(Hm, s) && intersects<W>(C[s], cmask); }, c2, nxt, L2, s2);
    }
    if (!found) return -1;
    if (lane == L2) M.assign(s2, cur);
    x[MS_AT(cur, N)] = (short)c2;
    set_bit<W>(changed, cur);
    hi = max(hi, cur);
    work[WK_AUG]++;
    if (lvl == 1) return 1;
    if (nxt < 0) return -1;
    cur = nxt;
    --lvl;
  }
  return -1;
}

// Time of one expert batch of g tokens (see moesched_model_t).
__device__ __forceinline__ long long batch_time_ns(const moesched_model_t& m, long long g) {
  if (g <= 0) return 0;
  const long long beyond = g > m.expert_knee_tokens ? g - m.expert_knee_tokens : 0;
  return m.expert_fixed_ns + (beyond * m.expert_ps_per_token + 999) / 1000;
}

// Division by a divisor fixed for the whole launch (the link speed): floor(x / d) for
// 0 <= x < 2^55 as a multiply-high and a shift (Granlund-Montgomery: with l = ceil(log2 d) and
// m = ceil(2^(55+l) / d), m*d lies in [2^(55+l), 2^(55+l) + 2^l], which makes the quotient exact
// for every 55-bit x).
struct FastDiv {
  unsigned long long m;
  int sh;
};
inline FastDiv make_fastdiv(long long d) {
  int l = 0;
  while ((1LL << l) < d) ++l;
  const unsigned __int128 num = (unsigned __int128)1 << (55 + l);
  FastDiv f;
  f.m = (unsigned long long)((num + (unsigned __int128)(d - 1)) / (unsigned __int128)d);
  f.sh = 55 + l;
  return f;
}
__device__ __forceinline__ long long fast_div(long long x, const FastDiv& f) {
  const unsigned long long hi = __umul64hi(f.m, (unsigned long long)x);
  const unsigned long long lo = f.m * (unsigned long long)x;
  return (long long)(f.sh >= 64 ? hi >> (f.sh - 64) : (hi << (64 - f.sh)) | (lo >> f.sh));
}

// ---- host-side launch geometry ---------------------------------------------------------------
struct Geometry {
  int cpl;       // columns per lane: 1, 2, 4 or 8
  int S;         // shared-memory row stride in ints
  bool cluster;  // matrix split over a 2-CTA cluster
  int wpb;       // warps (matrices) per CTA
  size_t smem;   // dynamic shared memory per CTA
};
Geometry plan_geometry(int N);
int sm_count();   // SMs of the current device (148 on B200), cached per device

cudaError_t run_mw(int B, int N, const int32_t* demand, int k_max, uint8_t* perm, int32_t* dur, int32_t* count,
                   int32_t* residual, int32_t* status, long long* work, cudaStream_t stream);
cudaError_t run_bvn(int B, int N, const int32_t* demand, int k_max, uint8_t* perm, int32_t* coef, int32_t* count,
                    int32_t* aug, int32_t* scratch, int32_t* status, long long* work, cudaStream_t stream);
// the same decomposition with one CTA of several warps per matrix (scratch required, 64 < N <= 256)
cudaError_t run_bvn_team(int B, int N, const int32_t* demand, int k_max, uint8_t* perm, int32_t* coef,
                         int32_t* count, int32_t* aug, int32_t* scratch, int32_t* status, long long* work,
                         cudaStream_t stream);
// row stride (ints) of the global working copy used by the Birkhoff kernel
inline int bvn_scratch_stride(int N) { return (N + 7) / 8 * 8; }
cudaError_t run_eval(int B, int N, const int32_t* demand, int k_stride, const uint8_t* perm, const int32_t* dur,
                     const int32_t* count, const moesched_model_t& model, long long* overlap, long long* serial,
                     long long* idle_ns, long long* idle_tok, long long* unserved, int32_t* status,
                     long long* prefix_overlap, long long* prefix_unserved, cudaStream_t stream, bool jobs = false);
// matching order and budget choice (order_kernel.cu)
cudaError_t run_order(int B, int k_stride, const long long* leg, const long long* comp, const int32_t* count,
                      const int32_t* eval_status, int32_t* order, long long* best_ns, long long* emission_ns,
                      int32_t* rule, int32_t* status, cudaStream_t stream);
cudaError_t run_permute(int B, int N, int k_stride, const uint8_t* perm, const int32_t* dur, const int32_t* order,
                        uint8_t* perm_out, int32_t* dur_out, cudaStream_t stream);
cudaError_t run_best_budget(int B, int k_stride, const int32_t* count, const long long* prefix_overlap,
                            const long long* prefix_unserved, long long price, int32_t* best_k, long long* best_cost,
                            cudaStream_t stream);

// greedy decomposition with one CTA per matrix, for the matrices whose status holds CLASS_U16 (64 < N <= 256)
cudaError_t run_mw_team(int B, int N, const int32_t* demand, int k_max, uint8_t* perm, int32_t* dur, int32_t* count,
                        int32_t* residual, int32_t* status, long long* work, cudaStream_t stream);

// scoring with one CTA per matrix, for the matrices whose status holds CLASS_U16 (64 < N <= 256)
cudaError_t run_eval_team(int B, int N, const int32_t* demand, int k_stride, const uint8_t* perm, const int32_t* dur,
                          const int32_t* count, const moesched_model_t& model, long long* overlap, long long* serial,
                          long long* idle_ns, long long* idle_tok, long long* unserved, int32_t* status,
                          cudaStream_t stream);

// class codes the pre-pass leaves in status[b] (never equal to a final status)
constexpr int CLASS_U16 = 64;
constexpr int CLASS_I32 = 65;
cudaError_t classify_matrices(int B, int N, const int32_t* demand, int32_t* status, cudaStream_t stream);

bool model_in_range(const moesched_model_t& m);
cudaError_t run_ideal_a2a(int B, int N, const int32_t* demand, const moesched_model_t& model, long long* comm_ns,
                          long long* makespan_ns, int32_t* status, cudaStream_t stream);

cudaError_t run_sinkhorn(int B, int N, const int32_t* demand, int iters, double smooth, int scale_bits,
                         double* scaled, int32_t* fixed, double* stretch, double* row_err, int32_t* status,
                         cudaStream_t stream);
cudaError_t run_sinkhorn_durations(int B, int k_stride, const int32_t* coef, const int32_t* count,
                                   const double* stretch, int scale_bits, int32_t* dur, cudaStream_t stream);

cudaError_t run_bvn_real(int B, int N, const double* matrix, double tol, int k_max, uint8_t* perm, double* lambda,
                         int32_t* count, double* sum_lambda, double* max_left, double* scratch, int32_t* status,
                         cudaStream_t stream);

// Launch helper shared by the three kernels.
template <typename Kernel, typename... Args>
cudaError_t launch_warp_kernel(Kernel kern, const Geometry& ge, int B, cudaStream_t stream, Args... args) {
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ge.smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(32 * ge.wpb);
  cfg.dynamicSmemBytes = ge.smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  if (ge.cluster) {
    cfg.gridDim = dim3(2 * B);
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  } else {
    cfg.gridDim = dim3((B + ge.wpb - 1) / ge.wpb);
  }
  return cudaLaunchKernelEx(&cfg, kern, args...);
}

}  // namespace moesched
