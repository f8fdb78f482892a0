// C ABI of the library: argument checks, launch geometry, error reporting.
#include <vector>

#include "common.cuh"

namespace moesched {

static thread_local int g_last_cuda_error = 0;
int& last_cuda_error_slot() { return g_last_cuda_error; }

// Shared memory one CTA may request on sm_100a (227 KB).
constexpr size_t SMEM_LIMIT = 227 * 1024;

Geometry plan_geometry(int N) {
  Geometry ge;
  ge.cpl = N <= 32 ? 1 : N <= 64 ? 2 : N <= 128 ? 4 : 8;
  ge.S = (N + ge.cpl - 1) / ge.cpl * ge.cpl;
  ge.cluster = false;
  size_t per_warp = warp_smem_bytes(N, ge.S, ge.cpl, false);
  if (per_warp > SMEM_LIMIT) {
    ge.cluster = true;
    per_warp = warp_smem_bytes(N, ge.S, ge.cpl, true);
  }
  // several small matrices share a CTA so that an SM can hold up to 64 warps
  ge.wpb = 1;
  if (!ge.cluster && N <= 32) ge.wpb = 4;
  ge.smem = per_warp * ge.wpb;
  return ge;
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

static int fail_cuda(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return MOESCHED_ECUDA;
}

bool model_in_range(const moesched_model_t& m) {
  const int64_t lim20 = 1LL << 20, lim30 = 1LL << 30, lim40 = 1LL << 40;
  return m.bytes_per_token >= 1 && m.bytes_per_token <= lim20 && m.link_gbps >= 1 && m.link_gbps <= lim20 &&
         m.reconfig_ns >= 0 && m.reconfig_ns <= lim40 && m.expert_fixed_ns >= 0 && m.expert_fixed_ns <= lim40 &&
         m.expert_ps_per_token >= 0 && m.expert_ps_per_token <= lim30 && m.expert_knee_tokens >= 0 &&
         m.expert_knee_tokens <= 2147483647LL;
}

#ifdef MOESCHED_CHECKED
static std::vector<FaultReader>& fault_readers() {
  static std::vector<FaultReader> readers;   // built on first use: the files register during static initialisation
  return readers;
}
void register_fault_reader(FaultReader reader) { fault_readers().push_back(reader); }
#endif

static bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3) == 0; }
static bool aligned8(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 7) == 0; }

}  // namespace moesched

using namespace moesched;

extern "C" {

int moesched_mw_decompose(int B, int N, const int32_t* d_demand, int k_max, uint8_t* d_perm, int32_t* d_dur,
                          int32_t* d_count, int32_t* d_residual, int32_t* d_status, int64_t* d_work,
                          void* stream) {
  if (B < 0 || N < 1 || N > MOESCHED_MAX_N || k_max < 1) return MOESCHED_EINVAL;
  if (B == 0) return MOESCHED_OK;
  if (!d_demand || !d_perm || !d_dur || !d_count || !d_status) return MOESCHED_EINVAL;
  if (!aligned4(d_demand) || !aligned4(d_dur) || !aligned4(d_count) || !aligned4(d_status) ||
      !aligned4(d_residual) || !aligned8(d_work))
    return MOESCHED_EINVAL;
  cudaError_t e = run_mw(B, N, d_demand, k_max, d_perm, d_dur, d_count, d_residual, d_status,
                         reinterpret_cast<long long*>(d_work), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOESCHED_OK : fail_cuda(e);
}

size_t moesched_bvn_scratch_bytes(int B, int N) {
  if (B < 0 || N < 1 || N > MOESCHED_MAX_N) return 0;
  return (size_t)B * N * bvn_scratch_stride(N) * sizeof(int32_t);
}

size_t moesched_workspace_bytes(int B, int N, int k_max) {
  if (k_max < 1) return 0;
  return moesched_bvn_scratch_bytes(B, N);
}

int moesched_bvn_decompose(int B, int N, const int32_t* d_demand, int k_max, uint8_t* d_perm, int32_t* d_coef,
                           int32_t* d_count, int32_t* d_aug, int32_t* d_scratch, int32_t* d_status,
                           int64_t* d_work, void* stream) {
  if (B < 0 || N < 1 || N > MOESCHED_MAX_N || k_max < 1) return MOESCHED_EINVAL;
  if (B == 0) return MOESCHED_OK;
  if (!d_demand || !d_perm || !d_coef || !d_count || !d_status) return MOESCHED_EINVAL;
  if (!aligned4(d_demand) || !aligned4(d_coef) || !aligned4(d_count) || !aligned4(d_status) || !aligned4(d_aug) ||
      !aligned8(d_work) || (reinterpret_cast<uintptr_t>(d_scratch) & 31) != 0)
    return MOESCHED_EINVAL;
  cudaError_t e = run_bvn(B, N, d_demand, k_max, d_perm, d_coef, d_count, d_aug, d_scratch, d_status,
                          reinterpret_cast<long long*>(d_work), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOESCHED_OK : fail_cuda(e);
}

static int schedule_eval_impl(int B, int N, const int32_t* d_demand, int k_stride, const uint8_t* d_perm,
                              const int32_t* d_dur, const int32_t* d_count, const moesched_model_t* h_model,
                              int64_t* d_makespan_overlap_ns, int64_t* d_makespan_serial_ns,
                              int64_t* d_compute_idle_ns, int64_t* d_link_idle_tokens, int64_t* d_unserved_tokens,
                              int32_t* d_status, int64_t* d_prefix_overlap_ns, int64_t* d_prefix_unserved_tokens,
                              void* stream) {
  if (B < 0 || N < 1 || N > MOESCHED_MAX_N || k_stride < 1) return MOESCHED_EINVAL;
  if (B == 0) return MOESCHED_OK;
  if (!d_demand || !d_perm || !d_dur || !d_count || !h_model || !d_makespan_overlap_ns ||
      !d_makespan_serial_ns || !d_compute_idle_ns || !d_link_idle_tokens || !d_unserved_tokens || !d_status)
    return MOESCHED_EINVAL;
  if (!aligned4(d_demand) || !aligned4(d_dur) || !aligned4(d_count) || !aligned4(d_status) ||
      !aligned8(d_makespan_overlap_ns) || !aligned8(d_makespan_serial_ns) || !aligned8(d_compute_idle_ns) ||
      !aligned8(d_link_idle_tokens) || !aligned8(d_unserved_tokens) || !aligned8(d_prefix_overlap_ns) ||
      !aligned8(d_prefix_unserved_tokens))
    return MOESCHED_EINVAL;
  const moesched_model_t m = *h_model;
  if (!model_in_range(m)) return MOESCHED_EINVAL;
  cudaError_t e = run_eval(B, N, d_demand, k_stride, d_perm, d_dur, d_count, m,
                           reinterpret_cast<long long*>(d_makespan_overlap_ns),
                           reinterpret_cast<long long*>(d_makespan_serial_ns),
                           reinterpret_cast<long long*>(d_compute_idle_ns),
                           reinterpret_cast<long long*>(d_link_idle_tokens),
                           reinterpret_cast<long long*>(d_unserved_tokens), d_status,
                           reinterpret_cast<long long*>(d_prefix_overlap_ns),
                           reinterpret_cast<long long*>(d_prefix_unserved_tokens),
                           static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOESCHED_OK : fail_cuda(e);
}

int moesched_schedule_eval(int B, int N, const int32_t* d_demand, int k_stride, const uint8_t* d_perm,
                           const int32_t* d_dur, const int32_t* d_count, const moesched_model_t* h_model,
                           int64_t* d_makespan_overlap_ns, int64_t* d_makespan_serial_ns,
                           int64_t* d_compute_idle_ns, int64_t* d_link_idle_tokens, int64_t* d_unserved_tokens,
                           int32_t* d_status, void* stream) {
  return schedule_eval_impl(B, N, d_demand, k_stride, d_perm, d_dur, d_count, h_model, d_makespan_overlap_ns,
                            d_makespan_serial_ns, d_compute_idle_ns, d_link_idle_tokens, d_unserved_tokens,
                            d_status, nullptr, nullptr, stream);
}

int moesched_schedule_prefix_eval(int B, int N, const int32_t* d_demand, int k_stride, const uint8_t* d_perm,
                                  const int32_t* d_dur, const int32_t* d_count, const moesched_model_t* h_model,
                                  int64_t* d_makespan_overlap_ns, int64_t* d_makespan_serial_ns,
                                  int64_t* d_compute_idle_ns, int64_t* d_link_idle_tokens,
                                  int64_t* d_unserved_tokens, int32_t* d_status, int64_t* d_prefix_overlap_ns,
                                  int64_t* d_prefix_unserved_tokens, void* stream) {
  if (B > 0 && (!d_prefix_overlap_ns || !d_prefix_unserved_tokens)) return MOESCHED_EINVAL;
  return schedule_eval_impl(B, N, d_demand, k_stride, d_perm, d_dur, d_count, h_model, d_makespan_overlap_ns,
                            d_makespan_serial_ns, d_compute_idle_ns, d_link_idle_tokens, d_unserved_tokens,
                            d_status, d_prefix_overlap_ns, d_prefix_unserved_tokens, stream);
}

size_t moesched_order_scratch_bytes(int B, int k_stride) {
  if (B < 0 || k_stride < 1 || k_stride > MOESCHED_ORDER_MAX_K) return 0;
  return (size_t)B * (2 * (size_t)k_stride + 5) * sizeof(int64_t) + (((size_t)B * sizeof(int32_t) + 7) & ~(size_t)7);
}

int moesched_schedule_order(int B, int N, const int32_t* d_demand, int k_stride, const uint8_t* d_perm,
                            const int32_t* d_dur, const int32_t* d_count, const moesched_model_t* h_model,
                            int32_t* d_order, int64_t* d_makespan_ns, int64_t* d_emission_ns, int32_t* d_rule,
                            int32_t* d_status, void* d_scratch, void* stream) {
  if (B < 0 || N < 1 || N > MOESCHED_MAX_N || k_stride < 1 || k_stride > MOESCHED_ORDER_MAX_K) return MOESCHED_EINVAL;
  if (B == 0) return MOESCHED_OK;
  if (!d_demand || !d_perm || !d_dur || !d_count || !h_model || !d_order || !d_makespan_ns || !d_emission_ns ||
      !d_rule || !d_status || !d_scratch)
    return MOESCHED_EINVAL;
  if (!aligned4(d_demand) || !aligned4(d_dur) || !aligned4(d_count) || !aligned4(d_order) || !aligned4(d_rule) ||
      !aligned4(d_status) || !aligned8(d_makespan_ns) || !aligned8(d_emission_ns) || !aligned8(d_scratch))
    return MOESCHED_EINVAL;
  const moesched_model_t m = *h_model;
  if (!model_in_range(m)) return MOESCHED_EINVAL;
  // scratch: job times [B][k_stride] x 2, five score arrays [B], the scoring status [B]
  long long* leg = static_cast<long long*>(d_scratch);
  long long* comp = leg + (size_t)B * k_stride;
  long long* scores = comp + (size_t)B * k_stride;
  int32_t* eval_status = reinterpret_cast<int32_t*>(scores + (size_t)5 * B);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = run_eval(B, N, d_demand, k_stride, d_perm, d_dur, d_count, m, scores, scores + B, scores + 2 * (size_t)B,
                           scores + 3 * (size_t)B, scores + 4 * (size_t)B, eval_status, leg, comp, st, true);
  if (e == cudaSuccess)
    e = run_order(B, k_stride, leg, comp, d_count, eval_status, d_order, reinterpret_cast<long long*>(d_makespan_ns),
                  reinterpret_cast<long long*>(d_emission_ns), d_rule, d_status, st);
  return e == cudaSuccess ? MOESCHED_OK : fail_cuda(e);
}

int moesched_schedule_permute(int B, int N, int k_stride, const uint8_t* d_perm, const int32_t* d_dur,
                              const int32_t* d_order, uint8_t* d_perm_out, int32_t* d_dur_out, void* stream) {
  if (B < 0 || N < 1 || N > MOESCHED_MAX_N || k_stride < 1) return MOESCHED_EINVAL;
  if (B == 0) return MOESCHED_OK;
  if (!d_perm || !d_dur || !d_order || !d_perm_out || !d_dur_out) return MOESCHED_EINVAL;
  if (!aligned4(d_dur) || !aligned4(d_order) || !aligned4(d_dur_out) || d_perm == d_perm_out || d_dur == d_dur_out)
    return MOESCHED_EINVAL;
  cudaError_t e = run_permute(B, N, k_stride, d_perm, d_dur, d_order, d_perm_out, d_dur_out,
                              static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOESCHED_OK : fail_cuda(e);
}

int moesched_best_budget(int B, int k_stride, const int32_t* d_count, const int64_t* d_prefix_overlap_ns,
                         const int64_t* d_prefix_unserved_tokens, int64_t ns_per_unserved_token,
                         int32_t* d_best_k, int64_t* d_best_cost, void* stream) {
  if (B < 0 || k_stride < 1 || ns_per_unserved_token < 0 || ns_per_unserved_token > (1LL << 15)) return MOESCHED_EINVAL;
  if (B == 0) return MOESCHED_OK;
  if (!d_count || !d_prefix_overlap_ns || !d_prefix_unserved_tokens || !d_best_k || !d_best_cost) return MOESCHED_EINVAL;
  if (!aligned4(d_count) || !aligned4(d_best_k) || !aligned8(d_prefix_overlap_ns) ||
      !aligned8(d_prefix_unserved_tokens) || !aligned8(d_best_cost))
    return MOESCHED_EINVAL;
  cudaError_t e = run_best_budget(B, k_stride, d_count, reinterpret_cast<const long long*>(d_prefix_overlap_ns),
                                  reinterpret_cast<const long long*>(d_prefix_unserved_tokens),
                                  (long long)ns_per_unserved_token, d_best_k,
                                  reinterpret_cast<long long*>(d_best_cost), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOESCHED_OK : fail_cuda(e);
}

int moesched_ideal_a2a(int B, int N, const int32_t* d_demand, const moesched_model_t* h_model, int64_t* d_comm_ns,
                       int64_t* d_makespan_ns, int32_t* d_status, void* stream) {
  if (B < 0 || N < 1 || N > MOESCHED_MAX_N) return MOESCHED_EINVAL;
  if (B == 0) return MOESCHED_OK;
  if (!d_demand || !h_model || !d_comm_ns || !d_makespan_ns || !d_status) return MOESCHED_EINVAL;
  if (!aligned4(d_demand) || !aligned4(d_status) || !aligned8(d_comm_ns) || !aligned8(d_makespan_ns))
    return MOESCHED_EINVAL;
  const moesched_model_t m = *h_model;
  if (!model_in_range(m)) return MOESCHED_EINVAL;
  cudaError_t e = run_ideal_a2a(B, N, d_demand, m, reinterpret_cast<long long*>(d_comm_ns),
                                reinterpret_cast<long long*>(d_makespan_ns), d_status,
                                static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOESCHED_OK : fail_cuda(e);
}

int moesched_sinkhorn_scale(int B, int N, const int32_t* d_demand, int iters, double smooth, int scale_bits,
                            double* d_scaled, int32_t* d_fixed, double* d_stretch, double* d_row_err,
                            int32_t* d_status, void* stream) {
  if (B < 0 || N < 1 || N > MOESCHED_MAX_N || iters < 1 || !(smooth >= 0.0) || scale_bits < 1 || scale_bits > 24)
    return MOESCHED_EINVAL;
  if (B == 0) return MOESCHED_OK;
  if (!d_demand || !d_scaled || !d_fixed || !d_stretch || !d_row_err || !d_status) return MOESCHED_EINVAL;
  if (!aligned4(d_demand) || !aligned4(d_fixed) || !aligned4(d_status) || !aligned8(d_scaled) ||
      !aligned8(d_stretch) || !aligned8(d_row_err))
    return MOESCHED_EINVAL;
  cudaError_t e = run_sinkhorn(B, N, d_demand, iters, smooth, scale_bits, d_scaled, d_fixed, d_stretch, d_row_err,
                               d_status, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOESCHED_OK : fail_cuda(e);
}

int moesched_sinkhorn_durations(int B, int k_stride, const int32_t* d_coef, const int32_t* d_count,
                                const double* d_stretch, int scale_bits, int32_t* d_dur, void* stream) {
  if (B < 0 || k_stride < 1 || scale_bits < 1 || scale_bits > 24) return MOESCHED_EINVAL;
  if (B == 0) return MOESCHED_OK;
  if (!d_coef || !d_count || !d_stretch || !d_dur) return MOESCHED_EINVAL;
  if (!aligned4(d_coef) || !aligned4(d_count) || !aligned4(d_dur) || !aligned8(d_stretch)) return MOESCHED_EINVAL;
  cudaError_t e = run_sinkhorn_durations(B, k_stride, d_coef, d_count, d_stretch, scale_bits, d_dur,
                                         static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOESCHED_OK : fail_cuda(e);
}

int moesched_bvn_real_decompose(int B, int N, const double* d_matrix, double tol, int k_max, uint8_t* d_perm,
                                double* d_lambda, int32_t* d_count, double* d_sum_lambda, double* d_max_left,
                                double* d_scratch, int32_t* d_status, void* stream) {
  if (B < 0 || N < 1 || N > MOESCHED_MAX_N || k_max < 1 || !(tol >= 0.0)) return MOESCHED_EINVAL;
  if (B == 0) return MOESCHED_OK;
  if (!d_matrix || !d_perm || !d_lambda || !d_count || !d_sum_lambda || !d_max_left || !d_scratch || !d_status)
    return MOESCHED_EINVAL;
  if (!aligned8(d_matrix) || !aligned8(d_lambda) || !aligned8(d_sum_lambda) || !aligned8(d_max_left) ||
      !aligned8(d_scratch) || !aligned4(d_count) || !aligned4(d_status))
    return MOESCHED_EINVAL;
  cudaError_t e = run_bvn_real(B, N, d_matrix, tol, k_max, d_perm, d_lambda, d_count, d_sum_lambda, d_max_left,
                               d_scratch, d_status, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOESCHED_OK : fail_cuda(e);
}

long long moesched_debug_index_faults(void) {
#ifdef MOESCHED_CHECKED
  if (cudaDeviceSynchronize() != cudaSuccess) return -2;
  long long total = 0;
  for (FaultReader read : fault_readers()) {
    const unsigned v = read();
    if (v == 0xffffffffu) return -2;
    total += v;
  }
  return total;
#else
  return -1;
#endif
}

int moesched_last_cuda_error(void) { return g_last_cuda_error; }

const char* moesched_strerror(int code) {
  switch (code) {
    case MOESCHED_OK: return "ok";
    case MOESCHED_EINVAL: return "invalid argument: null or misaligned pointer, or a size out of range";
    case MOESCHED_ECUDA: return "a CUDA call failed (see moesched_last_cuda_error)";
    case MOESCHED_ETOOBIG: return "batch too large for the library's built-in scratch array";
    default: return "unknown moesched return code";
  }
}

const char* moesched_status_str(int status) {
  switch (status) {
    case MOESCHED_ST_OK: return "ok: complete result";
    case MOESCHED_ST_TRUNCATED: return "truncated: the matching budget ran out before the matrix did";
    case MOESCHED_ST_BAD_INPUT: return "bad input: the matrix or schedule violates the documented range";
    case MOESCHED_ST_INTERNAL: return "internal: an iteration limit was hit (a bug in the library)";
    default: return "unknown moesched status";
  }
}

}  // extern "C"
