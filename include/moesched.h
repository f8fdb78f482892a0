/*
 * moesched -- batched circuit scheduling of MoE all-to-all demand matrices on
 * one NVIDIA B200 (sm_100a).
 *
 * For B independent N x N matrices of token counts (demand[b][i][j] = tokens
 * that rank i sends to rank j) the library computes, entirely on the GPU,
 *   - the greedy max-weight decomposition           (paper Sec. 3.2),
 *   - the Birkhoff-von Neumann decomposition        (paper Sec. 3.1),
 *   - the makespan of such a schedule under the dispatch -> expert compute ->
 *     combine pipeline with and without overlap     (paper Sec. 4.1, Sec. 3.3).
 *
 * Conventions shared by all entry points
 *   - Plain C ABI. Pointers named d_* are DEVICE pointers, h_* are HOST
 *     pointers. The caller owns every buffer; the library allocates nothing,
 *     frees nothing and never synchronises: work is enqueued on `stream`
 *     (a cudaStream_t passed as void*, NULL = default stream) and the call
 *     returns at once. Buffers must stay alive until the stream has drained.
 *   - Matrices are int32, row major, [B][N][N], densely packed. 1 <= N <= 256.
 *     d_demand should be 16-byte aligned (it then takes the bulk-copy path for
 *     even N; any 4-byte aligned pointer is still accepted).
 *   - A matching is a permutation pi stored as N bytes: pi[i] = destination
 *     rank of source rank i. Schedules are [B][k_max][N] uint8 plus
 *     [B][k_max] int32 durations (in tokens); only the first count[b]
 *     matchings of matrix b are written.
 *   - Tie rule: where several permutations are optimal the lexicographically
 *     smallest one is returned (row 0 gets the lowest column that any optimal
 *     matching allows, then row 1, ...). Results are therefore unique and
 *     independent of the solver.
 *   - Return value: MOESCHED_OK when the work was enqueued; MOESCHED_EINVAL
 *     for a null pointer or an out-of-range size (nothing enqueued); B = 0 is
 *     accepted, enqueues nothing and does not look at the pointers;
 *     MOESCHED_ECUDA when a CUDA call failed (moesched_last_cuda_error()).
 *   - d_status doubles as working memory while a call runs (from N = 48 up the greedy and
 *     scoring entry points park a per-matrix class code there between their kernels); it
 *     holds the outcome once the stream has passed the call.
 *   - Per-matrix outcome in d_status[b]:
 *       MOESCHED_ST_OK          complete result
 *       MOESCHED_ST_TRUNCATED   k_max matchings written, matrix not exhausted
 *       MOESCHED_ST_BAD_INPUT   matrix b violates the input range; count = 0
 *       MOESCHED_ST_INTERNAL    an internal iteration limit was hit (a bug)
 *     No input makes a kernel trap, spin or read out of bounds.
 */
#ifndef MOESCHED_H_
#define MOESCHED_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOESCHED_OK 0
#define MOESCHED_EINVAL (-1)
#define MOESCHED_ECUDA (-2)
#define MOESCHED_ETOOBIG (-3)

#define MOESCHED_ST_OK 0
#define MOESCHED_ST_TRUNCATED 1
#define MOESCHED_ST_BAD_INPUT (-1)
#define MOESCHED_ST_INTERNAL (-2)

#define MOESCHED_MAX_N 256

/* Largest entry the greedy decomposition accepts (2^28): its integer duals stay within a
 * few multiples of the largest entry, which must fit 31 bits. */
#define MOESCHED_MW_MAX_ENTRY 268435456

/* Number of int64 work counters per matrix written to d_work (see below). */
#define MOESCHED_WORK_FIELDS 10

/* Link and compute model of the overlap pipeline (paper Sec. 4.1 "Execution
 * time"): a matching lasts as long as its largest transfer at link speed; an
 * expert batch costs a fixed overhead plus a per-token cost (the affine form
 * of the "knee" of Fig. 1); circuits are reconfigured before every matching.
 * All integers. Ranges: 1 <= bytes_per_token <= 2^20, 1 <= link_gbps <= 2^20,
 * 0 <= reconfig_ns, expert_fixed_ns <= 2^40, 0 <= expert_ps_per_token <= 2^30,
 * 0 <= expert_knee_tokens <= 2^31-1.
 * Batch time of g > 0 tokens: expert_fixed_ns + ceil(max(0, g - expert_knee_tokens) *
 * expert_ps_per_token / 1000); 0 for g = 0. expert_knee_tokens = 0 is the affine model;
 * 250000 ns with a knee of 256 tokens are the constants the paper reports for its profiled
 * curve (Fig. 1, Sec. 3.1). */
typedef struct moesched_model {
  int64_t bytes_per_token;     /* payload of one routed token, bytes            */
  int64_t link_gbps;           /* port speed in Gb/s == bits per nanosecond     */
  int64_t reconfig_ns;         /* circuit reconfiguration delay per matching    */
  int64_t expert_fixed_ns;     /* fixed cost of one expert batch                */
  int64_t expert_ps_per_token; /* marginal cost per token, picoseconds          */
  int64_t expert_knee_tokens;  /* batch size up to which only the fixed cost is paid */
} moesched_model_t;

/*
 * Greedy max-weight decomposition (paper Sec. 3.2): a maximum-weight perfect
 * matching of what is left of the matrix is taken out again and again until
 * nothing is left, or until the budget k_max is used up.
 *
 * Per matrix: R <- D; while k < k_max and R != 0: pi_k <- lexicographically
 * smallest permutation maximising sum_i R[i][pi(i)] (zero entries are ordinary
 * weight-0 edges, so pi_k is always a full permutation); d_dur[b][k] <- largest
 * matched entry (paper Sec. 3.3 / 4.1: the heaviest pair sets the completion
 * time); the matched entries are served whole and set to zero.
 *
 *   d_demand   in   [B][N][N] int32, 0 <= entry <= MOESCHED_MW_MAX_ENTRY (2^28)
 *   k_max      in   matching budget and output capacity, >= 1
 *   d_perm     out  [B][k_max][N] uint8
 *   d_dur      out  [B][k_max] int32
 *   d_count    out  [B] int32 number of matchings written
 *   d_residual out  [B][N][N] int32 what is left of D (all zero unless
 *                   truncated); may be NULL
 *   d_status   out  [B] int32
 *   d_work     out  [B][MOESCHED_WORK_FIELDS] int64 work counters, may be NULL:
 *                   0 shortest-path column scans, 1 augmentations, 2 rows
 *                   tried against their best column, 3 canonicalisation
 *                   sweeps that searched, 4 search levels, 5 rotation steps,
 *                   6 matchings, 7 rows matched along tight edges before the
 *                   shortest-path phase, 8 rows expanded by the canonicalisation
 *                   searches (frontier pops), 9 groups of columns settled together
 *                   (CTA-per-matrix kernel only; there 0 counts the rows relaxed)
 */
int moesched_mw_decompose(int B, int N, const int32_t* d_demand, int k_max, uint8_t* d_perm,
                          int32_t* d_dur, int32_t* d_count, int32_t* d_residual,
                          int32_t* d_status, int64_t* d_work, void* stream);

/*
 * Birkhoff-von Neumann decomposition (paper Sec. 3.1: A = sum_k c_k P_k for a
 * matrix with equal row and column sums).
 *
 * The demand is first made balanced by an exact integer augmentation (the
 * paper names floating-point Sinkhorn-Knopp scaling as one possible
 * preprocessing; this library adds padding instead so that everything stays
 * integral): T = largest row or column sum; the deficits T - rowsum_i and
 * T - colsum_j are filled by the north-west-corner rule (lowest row first,
 * then lowest column), giving A = D + E with every row and column summing to
 * T and at most 2N-1 padded cells. Then, while A != 0 and k < k_max:
 * pi_k <- lexicographically smallest permutation with A[i][pi(i)] > 0 for all
 * i; c_k <- min_i A[i][pi_k(i)]; A <- A - c_k P_k. At most N^2 - 2N + 2
 * matchings result; pass that as k_max for a complete decomposition.
 *
 *   d_demand   in   [B][N][N] int32, entries >= 0, every row and column sum
 *                   <= 2^31-1
 *   d_perm     out  [B][k_max][N] uint8
 *   d_coef     out  [B][k_max] int32 coefficients c_k (tokens per pair)
 *   d_count    out  [B] int32
 *   d_aug      out  [B][N][N] int32 the balanced matrix A; may be NULL
 *   d_scratch  tmp  moesched_bvn_scratch_bytes(B, N) bytes of device memory, 32-byte
 *                   aligned, or NULL. With scratch the working copy of every matrix
 *                   lives there (it stays in L2) and shared memory is left for
 *                   bookkeeping, so several times more matrices are in flight per SM:
 *                   the fast path. Without it the matrix is held in shared memory
 *                   (a 2-CTA cluster for N > 232). Results are identical. Contents
 *                   are undefined afterwards; calls that overlap in time need
 *                   separate scratch.
 *   d_status   out  [B] int32
 *   d_work     out  [B][MOESCHED_WORK_FIELDS] int64, may be NULL: 0 levels of the
 *                   repair searches, 1 rows moved by the repairs, 2 rows re-matched
 *                   canonically at once, 3 canonicalisation sweeps that searched,
 *                   4 search levels, 5 rotation steps, 6 matchings, 7 rows
 *                   skipped as unchanged prefix, 8 rows expanded by the
 *                   canonicalisation searches (frontier pops), 9 re-matchings
 *                   that needed rows below the row whose entry vanished
 * A batch that is resident on the GPU all at once (from 12 matrices per SM up, with
 * scratch, without d_work) is launched with its warps pacing one another through a
 * 128 KB table built into the library (a warp that is ahead sleeps for a moment). This
 * changes timing only, never results; entries carry the launch's number, so calls that
 * overlap on one GPU merely ignore each other's entries.
 */
int moesched_bvn_decompose(int B, int N, const int32_t* d_demand, int k_max, uint8_t* d_perm,
                           int32_t* d_coef, int32_t* d_count, int32_t* d_aug, int32_t* d_scratch,
                           int32_t* d_status, int64_t* d_work, void* stream);

/* Bytes of scratch that moesched_bvn_decompose can use for B matrices of size N
 * (B * N * roundup(N, 8) * 4); 0 for sizes out of range. */
size_t moesched_bvn_scratch_bytes(int B, int N);

/* Device working memory, in bytes, that a pass of the whole path over B matrices of size N can
 * use beyond its inputs and outputs, whatever the budget k_max: the greedy decomposition and the
 * scoring keep their working state in shared memory and need none, so this is the scratch of the
 * Birkhoff-von Neumann decomposition (moesched_bvn_scratch_bytes). 0 for sizes out of range
 * (B < 0, N outside 1..256, k_max < 1). */
size_t moesched_workspace_bytes(int B, int N, int k_max);

/*
 * Score a schedule (paper Sec. 4.1 "Execution time": a matching completes after
 * its largest transfer, and the experts start on a matching as soon as its
 * dispatch is done, while the next matching is already being sent; Sec. 3.3:
 * dispatch, compute and combine form a three-machine flow shop; the panels of
 * Fig. 3 / Fig. 4 without overlap run every phase to completion).
 *
 * Per matrix, replaying matchings k = 0 .. count-1 against D:
 *   served_i = min(dur_k, Dres[i][pi_k(i)]); Dres -= served  (real tokens first)
 *   g_k = max_i served_i, s_k = sum_i served_i
 *   t_k    = ceil(dur_k * bytes_per_token * 8 / link_gbps)            [ns]
 *   comp_k = batch time of g_k tokens (see moesched_model_t)
 *   Dsp_k = Dsp_{k-1} + reconfig_ns + t_k
 *   Cmp_k = max(Dsp_k, Cmp_{k-1}) + comp_k
 *   Cmb_k = max(Cmp_k, Cmb_{k-1}) + reconfig_ns + t_k
 *   makespan_overlap = Cmb_K;  makespan_serial = sum_k (2 (reconfig_ns + t_k) + comp_k)
 *   compute_idle = (Cmp_K - Dsp_1) - sum_k comp_k   (0 if K = 0)
 *   link_idle_tokens = sum_k (N dur_k - s_k);  unserved_tokens = sum Dres
 *
 *   d_demand  in   [B][N][N] int32, entries >= 0
 *   k_stride  in   matchings allocated per matrix in d_perm / d_dur
 *   d_perm    in   [B][k_stride][N] uint8, each used row a permutation of 0..N-1
 *   d_dur     in   [B][k_stride] int32, >= 0, sum over k <= 2^40; the dispatch stage
 *                  (sum of reconfig_ns + t_k) and the expert batches (sum of comp_k) must each
 *                  stay within 2^60 ns, so that no makespan can wrap (BAD_INPUT otherwise)
 *   d_count   in   [B] int32, 0 <= count <= k_stride
 *   h_model   in   HOST pointer, read during the call
 *   d_*       out  [B] int64 each; zero when status is BAD_INPUT
 *   d_status  out  [B] int32 (OK or BAD_INPUT)
 */
int moesched_schedule_eval(int B, int N, const int32_t* d_demand, int k_stride,
                           const uint8_t* d_perm, const int32_t* d_dur, const int32_t* d_count,
                           const moesched_model_t* h_model, int64_t* d_makespan_overlap_ns,
                           int64_t* d_makespan_serial_ns, int64_t* d_compute_idle_ns,
                           int64_t* d_link_idle_tokens, int64_t* d_unserved_tokens,
                           int32_t* d_status, void* stream);

/*
 * moesched_schedule_eval plus the scores of every prefix of the schedule (paper Sec. 3.3 asks how
 * the ordering and number of matchings shape the makespan; a smaller greedy budget yields a prefix
 * of the complete schedule, so one decomposition with the largest budget and this call give the
 * whole budget sweep). For k < count[b]:
 *   d_prefix_overlap_ns[b][k]      = makespan_overlap of matchings 0..k alone (= Cmb_{k+1})
 *   d_prefix_unserved_tokens[b][k] = tokens of D not yet served after matchings 0..k
 * Entries with k >= count[b], and all entries of a schedule flagged BAD_INPUT, are -1.
 * Both arrays are [B][k_stride] int64 device memory; all other arguments as in
 * moesched_schedule_eval.
 */
int moesched_schedule_prefix_eval(int B, int N, const int32_t* d_demand, int k_stride,
                                  const uint8_t* d_perm, const int32_t* d_dur, const int32_t* d_count,
                                  const moesched_model_t* h_model, int64_t* d_makespan_overlap_ns,
                                  int64_t* d_makespan_serial_ns, int64_t* d_compute_idle_ns,
                                  int64_t* d_link_idle_tokens, int64_t* d_unserved_tokens,
                                  int32_t* d_status, int64_t* d_prefix_overlap_ns,
                                  int64_t* d_prefix_unserved_tokens, void* stream);

/*
 * Order of the matchings (paper Sec. 3.3, last paragraph: dispatch, expert compute and combine are
 * the three machines of a flow shop and the order of the matchings changes the makespan; the paper
 * leaves the rule open). This entry point chooses the best of five orders on FIXED job times
 *   a_k = reconfig_ns + t_k (dispatch; the combine stage takes the same time),  b_k = comp_k,
 * both as the replay in emission order gives them (see moesched_schedule_eval). Candidates, ties
 * always by the lower original index: 0 the emission order; 1 Johnson's rule on stages one and two
 * (jobs with a <= b first by increasing a, then the rest by decreasing b); 2 Johnson's rule on stages
 * two and three (b <= a first by increasing b, then the rest by decreasing a); 3 increasing a, placed
 * alternately at the front and at the back (the shortest transfers open and close the schedule);
 * 4 decreasing b. Each is run through the three-stage recurrence; the shortest wins, the lower rule
 * number on ties, so the result is never worse than the emission order. The fixed times are exact
 * for the reordered schedule when no pair with demand occurs in two matchings; a greedy schedule
 * repeats a pair only as an idle filler, and scoring the reordered schedule (moesched_schedule_permute,
 * then moesched_schedule_eval) gives the exact figure where it matters.
 *
 *   k_stride          in   1 .. MOESCHED_ORDER_MAX_K
 *   d_demand ... h_model   as in moesched_schedule_eval
 *   d_order           out  [B][k_stride] int32: d_order[b][p] = original index of the matching that
 *                          runs at position p; -1 for p >= count[b] and for rejected schedules
 *   d_makespan_ns     out  [B] int64 makespan of the chosen order on the fixed job times
 *   d_emission_ns     out  [B] int64 the same for the emission order (= makespan_overlap_ns)
 *   d_rule            out  [B] int32 number of the winning candidate
 *   d_status          out  [B] int32 OK, or BAD_INPUT (a schedule moesched_schedule_eval rejects)
 *   d_scratch         tmp  moesched_order_scratch_bytes(B, k_stride) bytes, 8-byte aligned
 */
#define MOESCHED_ORDER_MAX_K 1024
size_t moesched_order_scratch_bytes(int B, int k_stride);
int moesched_schedule_order(int B, int N, const int32_t* d_demand, int k_stride, const uint8_t* d_perm,
                            const int32_t* d_dur, const int32_t* d_count, const moesched_model_t* h_model,
                            int32_t* d_order, int64_t* d_makespan_ns, int64_t* d_emission_ns, int32_t* d_rule,
                            int32_t* d_status, void* d_scratch, void* stream);

/* The schedule in a new order: d_perm_out[b][p] = d_perm[b][d_order[b][p]] and the same for the
 * durations, for every position whose order entry lies in 0 .. k_stride-1; other positions are left
 * untouched. The output arrays must not overlap the input arrays. */
int moesched_schedule_permute(int B, int N, int k_stride, const uint8_t* d_perm, const int32_t* d_dur,
                              const int32_t* d_order, uint8_t* d_perm_out, int32_t* d_dur_out, void* stream);

/*
 * Budget choice (paper Sec. 3.2 / 3.3: how many matchings are worth running): from the prefix scores of
 * moesched_schedule_prefix_eval and a price in ns per token left unserved (0 .. 2^15), the number of
 * matchings k in 1 .. count[b] that minimises
 *   d_prefix_overlap_ns[b][k-1] + ns_per_unserved_token * d_prefix_unserved_tokens[b][k-1],
 * the smallest such k on ties. d_best_k [B] int32, d_best_cost [B] int64; both 0 for an empty
 * schedule or one whose prefix entries are -1 (rejected).
 */
int moesched_best_budget(int B, int k_stride, const int32_t* d_count, const int64_t* d_prefix_overlap_ns,
                         const int64_t* d_prefix_unserved_tokens, int64_t ns_per_unserved_token,
                         int32_t* d_best_k, int64_t* d_best_cost, void* stream);

/*
 * Idealised congestion-free all-to-all (paper Sec. 4.1 "Comparisons": the best completion time
 * any fabric could reach for the matrix), the yardstick the decomposed schedules are compared
 * with. Every port sends and receives at line rate, so one exchange
 * lasts as long as its busiest port; dispatch, expert compute (all tokens of a rank in one
 * batch) and combine run to completion one after the other; no circuit is reconfigured.
 *   port_b  = max(largest row sum, largest column sum) of matrix b
 *   comm_ns = ceil(port_b * bytes_per_token * 8 / link_gbps)
 *   makespan_ns = 2 * comm_ns + batch time of the largest column sum
 *
 *   d_demand       in   [B][N][N] int32, entries >= 0, row and column sums <= 2^31-1
 *   h_model        in   HOST pointer, read during the call
 *   d_comm_ns      out  [B] int64
 *   d_makespan_ns  out  [B] int64
 *   d_status       out  [B] int32 (OK, or BAD_INPUT with both outputs 0)
 */
int moesched_ideal_a2a(int B, int N, const int32_t* d_demand, const moesched_model_t* h_model,
                       int64_t* d_comm_ns, int64_t* d_makespan_ns, int32_t* d_status, void* stream);

/*
 * Sinkhorn-Knopp scaling: the preprocessing the paper names for the Birkhoff-von Neumann
 * decomposition (Sec. 3.1: demand matrices are not doubly stochastic, so they are normalised
 * first; the normalisation moves mass between rows and columns and thereby adds capacity that
 * no routed token asked for). moesched_bvn_decompose pads instead; this entry point gives the paper's
 * multiplicative route: scale here, then decompose d_fixed with moesched_bvn_decompose, turn
 * its coefficients into token counts with moesched_sinkhorn_durations, and score the result
 * against the ORIGINAL demand with moesched_schedule_eval.
 *
 * The paper fixes no constants; the steps are: X = D + smooth; one sweep divides every entry of
 * X by the sum of its row and then every entry by the sum of its column; `iters` sweeps. IEEE
 * double arithmetic, row sums accumulated left to right and column sums top to
 * bottom, one rounding per operation -- the result is therefore reproducible bit for bit.
 *   d_scaled[b]  = X after the last sweep (column sums 1 up to rounding)
 *   d_row_err[b] = max_i |sum_j scaled[b][i][j] - 1|, the distance from double stochasticity
 *   d_fixed[b]   = floor(scaled * 2^scale_bits + 0.5), the integer matrix for the exact
 *                  decomposition (its padding absorbs the rounding residue)
 *   d_stretch[b] = max over pairs with D_ij > 0 and fixed_ij > 0 of D_ij * 2^scale_bits / fixed_ij:
 *                  tokens per unit of the scaled schedule such that every such pair can send all of
 *                  its demand; pairs that the balancing scaled up finish early and idle
 *   d_status[b]  = OK; TRUNCATED when a pair with demand was rounded to zero (it cannot be served);
 *                  BAD_INPUT for a negative entry or a row or column without mass (possible only
 *                  with smooth = 0): all outputs of that matrix are then 0.
 *
 *   d_demand   in   [B][N][N] int32, entries >= 0
 *   iters      in   number of sweeps, >= 1
 *   smooth     in   >= 0, added to every entry (gives empty rows and columns mass)
 *   scale_bits in   1..24
 *   d_scaled   out  [B][N][N] double, 8-byte aligned; also the working memory of the call
 *   d_fixed    out  [B][N][N] int32
 *   d_stretch, d_row_err  out  [B] double;  d_status  out  [B] int32
 */
int moesched_sinkhorn_scale(int B, int N, const int32_t* d_demand, int iters, double smooth, int scale_bits,
                            double* d_scaled, int32_t* d_fixed, double* d_stretch, double* d_row_err,
                            int32_t* d_status, void* stream);

/*
 * Length in tokens of every matching of a decomposition of d_fixed (paper Sec. 3.1: a matching
 * with coefficient lambda occupies that share of the scaled schedule):
 *   d_dur[b][k] = min(2^31-1, ceil(d_coef[b][k] * d_stretch[b] / 2^scale_bits))  for k < d_count[b],
 * in double arithmetic (one rounding in the product; the division by a power of two is exact).
 * Entries with k >= d_count[b] are left untouched. All arrays are device memory:
 * d_coef, d_dur [B][k_stride] int32, d_count [B] int32, d_stretch [B] double.
 */
int moesched_sinkhorn_durations(int B, int k_stride, const int32_t* d_coef, const int32_t* d_count,
                                const double* d_stretch, int scale_bits, int32_t* d_dur, void* stream);

/*
 * Birkhoff-von Neumann decomposition of a real-valued matrix (paper Sec. 3.1: A = sum_k lambda_k P_k
 * for a doubly stochastic A; Sec. 4.2 discusses the size of its coefficients). The usual input is
 * d_scaled of moesched_sinkhorn_scale, which is doubly stochastic only up to the error of its last
 * sweep; so entries at or below `tol` count as zero (on input and after every subtraction) and the
 * loop also ends when the support has no perfect matching left. Per step: pi_k = lexicographically
 * smallest permutation with positive entries, lambda_k = its smallest entry, subtracted along pi_k.
 * Single IEEE double operations in a fixed order: results are reproducible bit for bit.
 *
 *   d_matrix     in   [B][N][N] double, entries >= 0 (a negative or NaN entry: BAD_INPUT)
 *   tol          in   >= 0
 *   k_max        in   output capacity, >= 1 (N^2 - 2N + 2 always suffices)
 *   d_perm       out  [B][k_max][N] uint8
 *   d_lambda     out  [B][k_max] double coefficients
 *   d_count      out  [B] int32
 *   d_sum_lambda out  [B] double: ((lambda_0 + lambda_1) + ...), 1 up to what is left for a scaled matrix
 *   d_max_left   out  [B] double: the largest entry remaining when the loop ended
 *   d_scratch    tmp  B * N * roundup(N, 8) doubles, 8-byte aligned: the working copy
 *   d_status     out  [B] int32: OK (nothing left), TRUNCATED (entries left: no perfect matching any
 *                     more, or k_max reached), BAD_INPUT (count 0)
 */
int moesched_bvn_real_decompose(int B, int N, const double* d_matrix, double tol, int k_max, uint8_t* d_perm,
                                double* d_lambda, int32_t* d_count, double* d_sum_lambda, double* d_max_left,
                                double* d_scratch, int32_t* d_status, void* stream);

/*
 * Birkhoff-von Neumann decomposition for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of moesched_bvn_decompose,
 * same arguments, same results, minus d_scratch.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a framework that
 * owns the whole memory pool and hands out no raw allocations, in a plug-in or callback
 * that must not touch the allocator, or in a latency-critical loop where an allocation
 * (which may synchronise the device) is not acceptable. Such a caller passes inputs and
 * outputs it already has and still gets the fast path, because the working copy of the
 * matrices lives in an array built into the library: MOESCHED_STATIC_SCRATCH_BYTES of
 * device memory that every GPU using the library gives up from load until process exit.
 *
 * Limit: B * N * roundup(N, 8) * 4 bytes must not exceed MOESCHED_STATIC_SCRATCH_BYTES
 * (e.g. B <= 1024 at N = 64, B <= 64 at N = 256); larger batches return MOESCHED_ETOOBIG
 * and enqueue nothing -- split the batch or use moesched_bvn_decompose with your own scratch.
 *
 * The first call on each device looks up the array's device address (no allocation, but
 * a runtime query): make that first call with the device current and outside any stream
 * capture. The address is remembered per device for the life of the process; a caller that
 * resets the device (cudaDeviceReset) afterwards must not call this entry point again,
 * because the remembered address then points into a context that no longer exists.
 * All calls of one process on one GPU share the one array (another process has its own copy);
 * it holds whatever the previous call left and is fully rewritten for the rows it uses, so
 * nothing needs clearing, but two calls that can run at the same time on one GPU (from
 * different streams or threads of the process) would trample each other's working copy:
 * serialise them. No cudaMalloc, cudaFree or other allocating call is made.
 */
#define MOESCHED_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u)
int moesched_bvn_decompose_static(int B, int N, const int32_t* d_demand, int k_max, uint8_t* d_perm,
                                  int32_t* d_coef, int32_t* d_count, int32_t* d_aug,
                                  int32_t* d_status, int64_t* d_work, void* stream);

/*
 * Measurement aid (no counterpart in the paper): enqueue a kernel of `blocks` CTAs of 256
 * threads, each thread running 8 independent chains of add / min / xor for `iters`
 * iterations, and return the number of integer lane-operations it executes
 * (blocks * 256 * iters * 24), or a negative MOESCHED_* code. Timing the launch gives the
 * integer issue rate the decomposition kernels are measured against. d_out: device,
 * blocks * 256 uint32 (written so that the work cannot be optimised away).
 */
long long moesched_probe_int_ops(int blocks, int iters, uint32_t* d_out, void* stream);

/*
 * Debugging aid (no counterpart in the paper). The library can be built with -DMOESCHED_CHECKED
 * (paper_2605_26845_b200/build.py builds that variant as libmoesched_checked.so): every memory index
 * that the kernels derive from the matching state is then range-checked, an index out of range is
 * counted and replaced by 0 (the access stays in bounds, the kernel ends normally), and this call
 * returns how many were counted on the current device since the library was loaded. It
 * synchronises the device. A library built without the checks returns -1; -2 means a CUDA call
 * failed. Results of the checked build are identical to the normal one; it is slower.
 */
long long moesched_debug_index_faults(void);

/* CUDA error code (cudaError_t as int) of the last failed CUDA call made by
 * this library on the calling thread; 0 if none. */
int moesched_last_cuda_error(void);

/* Text for a MOESCHED_* RETURN CODE of an entry point (MOESCHED_OK, _EINVAL, _ECUDA, _ETOOBIG).
 * Never NULL. Per-matrix statuses share small numbers with the return codes and have their own
 * function below. */
const char* moesched_strerror(int code);

/* Text for a per-matrix MOESCHED_ST_* value read from a d_status array. Never NULL. */
const char* moesched_status_str(int status);

#ifdef __cplusplus
}
#endif
#endif /* MOESCHED_H_ */
