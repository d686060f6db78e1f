// extern "C" entry points of libatgrpo: argument validation, workspace carving, launch order.
#include "internal.h"

using namespace atgrpo;

namespace {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int64_t padded_rows(int64_t T, int M) {
  // every head occupies whole 256-row tiles (the row extent of a CTA pair)
  const int64_t tiles = (T + 255) / 256 + (M > 1 ? M : 0);
  return tiles * 256;
}

int sm_count_or_default() {
  int n_sm = 148, cc = 0;
  if (device_sm_count(&n_sm, &cc) != ATGRPO_OK || n_sm <= 0) n_sm = 148;
  return n_sm;
}

// Workspace layout shared by the forward and the backward call.
struct PolicyPlan {
  size_t sched, tok_of_row, row_of_token, routing, Hs, coef, gemm, loss, total;
  int64_t T_pad;
};
PolicyPlan policy_plan(int64_t T, int d, int V, int M, bool is_bwd, bool dH_direct, int n_sm) {
  PolicyPlan p;
  p.T_pad = padded_rows(T, M);
  Carver c(nullptr);
  p.sched = c.off; c.take<Schedule>(1);
  p.tok_of_row = c.off; c.take<int32_t>((size_t)p.T_pad);
  p.row_of_token = c.off; c.take<int32_t>((size_t)T + 1);
  p.routing = c.off; c.off += align_up(routing_workspace_bytes(T, M), 256);
  p.Hs = c.off;
  if (M > 1 || is_bwd) c.take<uint16_t>((size_t)p.T_pad * d);   // backward always gathers the rows it keeps
  p.coef = c.off;
  if (is_bwd) c.take<float>((size_t)T + 1);
  p.gemm = c.off;
  c.off += align_up(is_bwd ? lm_head_bwd_workspace_bytes(p.T_pad, d, V, dH_direct)
                           : lm_head_fwd_workspace_bytes(p.T_pad, d, V, n_sm), 256);
  p.loss = c.off;
  c.off += align_up(loss_reduce_workspace_bytes(T), 256);
  p.total = c.off;
  return p;
}

int policy_common_checks(const void* H, int64_t ldH, const void* const* W, int32_t M,
                         const int32_t* target, const int32_t* role_of_token,
                         const int32_t* head_of_role, int32_t n_role, const int32_t* resp_of_token,
                         const float* adv, int64_t n_resp, const float* old_logp, int64_t T,
                         int32_t d, int32_t V, const atgrpo_params* params, void* workspace) {
  if (!params_ok(params)) return ATGRPO_ERR_INVALID_ARG;
  if (T < 0 || n_resp < 0 || V < 1 || d < 1 || M < 1 || W == nullptr) return ATGRPO_ERR_INVALID_ARG;
  if (M > ATGRPO_MAX_HEADS || d % 8 != 0 || d < 64 || T >= 2147483647ll - 65536) return ATGRPO_ERR_UNSUPPORTED;
  if (ldH < d || ldH % 8 != 0) return ATGRPO_ERR_INVALID_ARG;
  for (int m = 0; m < M; ++m)
    if (W[m] == nullptr || !aligned(W[m], 16)) return ATGRPO_ERR_INVALID_ARG;
  if (T > 0) {
    if (H == nullptr || target == nullptr || resp_of_token == nullptr || adv == nullptr ||
        old_logp == nullptr)
      return ATGRPO_ERR_INVALID_ARG;
    if (!aligned(H, 16)) return ATGRPO_ERR_INVALID_ARG;
    if (M > 1 && (role_of_token == nullptr || head_of_role == nullptr || n_role < 1))
      return ATGRPO_ERR_INVALID_ARG;
  }
  if (workspace == nullptr || !aligned(workspace, 256)) return ATGRPO_ERR_WORKSPACE;
  if (params->logits != nullptr &&
      (!aligned(params->logits, 256) || params->logits_bytes < lm_head_logits_bytes(T, V, params->logits_format)))
    return ATGRPO_ERR_INVALID_ARG;
  return ATGRPO_OK;
}

// Shared body of atgrpo_policy_loss_bwd and atgrpo_policy_loss_bwd_notify (defined further down).
int policy_loss_bwd_impl(const void* H, int64_t ldH, const void* const* W, int32_t M,
                         const int32_t* target, const int32_t* role_of_token,
                         const int32_t* head_of_role, int32_t n_role,
                         const int32_t* resp_of_token, const float* adv, int64_t n_resp,
                         const float* old_logp, const float* logp, const float* lse,
                         const float* grad_loss, int64_t T, int32_t d, int32_t V,
                         const atgrpo_params* params, void* dH, void* const* dW,
                         void* const* chunk_events, int32_t n_events, bool notify,
                         int32_t* device_status, void* workspace, size_t workspace_bytes,
                         void* stream);

}  // namespace

extern "C" {

const char* atgrpo_status_string(int status) {
  switch (status) {
    case ATGRPO_OK: return "ok";
    case ATGRPO_ERR_INVALID_ARG: return "invalid argument";
    case ATGRPO_ERR_UNSUPPORTED: return "unsupported size or device";
    case ATGRPO_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case ATGRPO_ERR_BAD_INDEX: return "index out of range (detected on the device)";
    case ATGRPO_ERR_TIMEOUT: return "bounded wait expired inside a kernel";
    case ATGRPO_ERR_CUDA: return "CUDA call failed";
    case ATGRPO_ERR_LAYOUT: return "candidates_grouped was set but a group's members are not adjacent";
    default: return "unknown status";
  }
}

size_t atgrpo_group_advantages_workspace_bytes(int64_t n_cand, int64_t n_groups) {
  return group_adv_workspace_bytes(n_cand, n_groups);
}

int atgrpo_group_advantages(const float* rewards, const int32_t* env_id, const int32_t* role_id,
                            const int32_t* turn_id, int64_t n_cand, int32_t n_env, int32_t n_role,
                            int32_t n_turn, const atgrpo_params* params, float* adv,
                            int32_t* group_of_cand, int32_t* group_offsets, int32_t* group_perm,
                            float* group_mean, float* group_std, int32_t* device_status,
                            void* workspace, size_t workspace_bytes, void* stream) {
  if (!params_ok(params)) return ATGRPO_ERR_INVALID_ARG;
  if (n_cand < 0 || n_env < 1 || n_role < 1 || n_turn < 1) return ATGRPO_ERR_INVALID_ARG;
  const int64_t G = (int64_t)n_env * n_role * n_turn;
  if (G >= 2147483647ll || n_cand >= 2147483647ll) return ATGRPO_ERR_UNSUPPORTED;
  if (n_cand > 0 && (rewards == nullptr || env_id == nullptr || role_id == nullptr ||
                     turn_id == nullptr || adv == nullptr))
    return ATGRPO_ERR_INVALID_ARG;
  if (workspace == nullptr || !aligned(workspace, 256) ||
      workspace_bytes < group_adv_workspace_bytes(n_cand, G))
    return ATGRPO_ERR_WORKSPACE;
  return group_adv_launch(rewards, env_id, role_id, turn_id, n_cand, n_env, n_role, n_turn, *params,
                          adv, group_of_cand, group_offsets, group_perm, group_mean, group_std,
                          device_status, workspace, static_cast<cudaStream_t>(stream));
}

int atgrpo_group_advantages_packed(const float* rewards, const int32_t* group_id, int64_t n_cand,
                                   int64_t n_groups, const atgrpo_params* params, float* adv,
                                   int32_t* group_offsets, int32_t* group_perm, float* group_mean,
                                   float* group_std, int32_t* device_status, void* workspace,
                                   size_t workspace_bytes, void* stream) {
  if (!params_ok(params)) return ATGRPO_ERR_INVALID_ARG;
  if (n_cand < 0 || n_groups < 1) return ATGRPO_ERR_INVALID_ARG;
  if (n_groups >= 2147483647ll || n_cand >= 2147483647ll) return ATGRPO_ERR_UNSUPPORTED;
  if (n_cand > 0 && (rewards == nullptr || group_id == nullptr || adv == nullptr)) return ATGRPO_ERR_INVALID_ARG;
  if (workspace == nullptr || !aligned(workspace, 256) ||
      workspace_bytes < group_adv_workspace_bytes(n_cand, n_groups))
    return ATGRPO_ERR_WORKSPACE;
  return group_adv_launch(rewards, group_id, nullptr, nullptr, n_cand, (int32_t)n_groups, 1, 1, *params, adv,
                          nullptr, group_offsets, group_perm, group_mean, group_std, device_status, workspace,
                          static_cast<cudaStream_t>(stream), nullptr, true);
}

size_t atgrpo_group_select_workspace_bytes(int64_t n_cand, int64_t n_groups) {
  return group_select_workspace_bytes(n_cand, n_groups);
}

int atgrpo_group_select(const float* r_team, const float* r_loc, float alpha, const int32_t* env_id,
                        const int32_t* role_id, const int32_t* turn_id, int64_t n_cand, int32_t n_env,
                        int32_t n_role, int32_t n_turn, const atgrpo_params* params, float* rewards_out,
                        float* adv, int32_t* group_best, int32_t* group_of_cand, float* group_mean,
                        float* group_std, int32_t* device_status, void* workspace, size_t workspace_bytes,
                        void* stream) {
  if (!params_ok(params)) return ATGRPO_ERR_INVALID_ARG;
  if (n_cand < 0 || n_env < 1 || n_role < 1 || n_turn < 1) return ATGRPO_ERR_INVALID_ARG;
  const int64_t G = (int64_t)n_env * n_role * n_turn;
  if (G >= 2147483647ll || n_cand >= 2147483647ll) return ATGRPO_ERR_UNSUPPORTED;
  if (n_cand > 0 && (r_team == nullptr || r_loc == nullptr || env_id == nullptr || role_id == nullptr ||
                     turn_id == nullptr || adv == nullptr))
    return ATGRPO_ERR_INVALID_ARG;
  if (workspace == nullptr || !aligned(workspace, 256) ||
      workspace_bytes < group_select_workspace_bytes(n_cand, G))
    return ATGRPO_ERR_WORKSPACE;
  GroupExtras ex{r_team, r_loc, alpha, rewards_out, group_best};
  return group_adv_launch(nullptr, env_id, role_id, turn_id, n_cand, n_env, n_role, n_turn, *params, adv,
                          group_of_cand, nullptr, nullptr, group_mean, group_std, device_status, workspace,
                          static_cast<cudaStream_t>(stream), &ex);
}

size_t atgrpo_clipped_loss_workspace_bytes(int64_t T) { return loss_reduce_workspace_bytes(T); }

int atgrpo_clipped_loss(const float* logp, const float* old_logp, const int32_t* resp_of_token,
                        const float* adv, int64_t T, int64_t n_resp, const atgrpo_params* params,
                        float* loss, float* coef, int64_t* clip_counts, int32_t* device_status,
                        void* workspace, size_t workspace_bytes, void* stream) {
  if (!params_ok(params) || T < 0 || n_resp < 0 || loss == nullptr) return ATGRPO_ERR_INVALID_ARG;
  if (T > 0 && (logp == nullptr || old_logp == nullptr || resp_of_token == nullptr || adv == nullptr))
    return ATGRPO_ERR_INVALID_ARG;
  if (workspace == nullptr || !aligned(workspace, 256) ||
      workspace_bytes < loss_reduce_workspace_bytes(T))
    return ATGRPO_ERR_WORKSPACE;
  return loss_reduce_launch(logp, old_logp, resp_of_token, adv, n_resp, nullptr, nullptr, 0, 1, T,
                            *params, nullptr, loss, coef, clip_counts, device_status, workspace,
                            static_cast<cudaStream_t>(stream));
}

size_t atgrpo_policy_loss_workspace_bytes(int64_t T, int32_t d, int32_t V, int32_t M, int32_t is_bwd) {
  if (T < 0 || d < 1 || V < 1 || M < 1) return 0;
  // the backward plan is sized for the larger case (dH accumulated in the workspace)
  return policy_plan(T, d, V, M, is_bwd != 0, false, sm_count_or_default()).total;
}

size_t atgrpo_policy_loss_logits_bytes(int64_t T, int32_t V, int32_t logits_format) {
  if (T < 0 || V < 1 || (logits_format != ATGRPO_LOGITS_F32 && logits_format != ATGRPO_LOGITS_Q16)) return 0;
  return lm_head_logits_bytes(T, V, logits_format);
}

int32_t atgrpo_policy_loss_launch_count(int64_t T, int32_t d, int32_t V, int32_t M, int32_t is_bwd) {
  if (T <= 0 || d < 1 || V < 1 || M < 1) return 0;
  const int route = M == 1 ? 1 : 3;                  // single-head table, or histogram + scan + scatter
  if (!is_bwd) return route + (M > 1 ? 1 : 0) + 3;   // (+ row gather) + GEMM sweep, logsumexp combine, Eq. 2 reduction
  // routing for the counts, coef, routing of the gradient-carrying tokens, row gather,
  // one GEMM launch per vocabulary chunk plus one, dH cast
  return route + 1 + 3 + 1 + lm_head_bwd_chunks(padded_rows(T, M), d, V) + 1 + 1;
}

int atgrpo_policy_loss_fwd(const void* H, int64_t ldH, const void* const* W, int32_t M,
                           const int32_t* target, const int32_t* role_of_token,
                           const int32_t* head_of_role, int32_t n_role,
                           const int32_t* resp_of_token, const float* adv, int64_t n_resp,
                           const float* old_logp, int64_t T, int32_t d, int32_t V,
                           const atgrpo_params* params, float* loss, float* logp, float* lse,
                           int32_t* role_offsets, int32_t* role_perm, int64_t* clip_counts,
                           int32_t* device_status, void* workspace, size_t workspace_bytes,
                           void* stream) {
  int rc = policy_common_checks(H, ldH, W, M, target, role_of_token, head_of_role, n_role,
                                resp_of_token, adv, n_resp, old_logp, T, d, V, params, workspace);
  if (rc != ATGRPO_OK) return rc;
  if (loss == nullptr || (T > 0 && (logp == nullptr || lse == nullptr))) return ATGRPO_ERR_INVALID_ARG;
  int n_sm = 0, cc = 0;
  if (device_sm_count(&n_sm, &cc) != ATGRPO_OK) return ATGRPO_ERR_CUDA;
  if (cc != 10) return ATGRPO_ERR_UNSUPPORTED;
  const PolicyPlan pl = policy_plan(T, d, V, M, false, false, n_sm);
  if (workspace_bytes < pl.total) return ATGRPO_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  if (T == 0) {
    ATGRPO_CUDA_OK(cudaMemsetAsync(loss, 0, sizeof(float) * M, st));
    if (role_offsets) ATGRPO_CUDA_OK(cudaMemsetAsync(role_offsets, 0, sizeof(int32_t) * (M + 1), st));
    if (clip_counts) ATGRPO_CUDA_OK(cudaMemsetAsync(clip_counts, 0, sizeof(int64_t) * 2 * M, st));
    return ATGRPO_OK;
  }
  Schedule* sched = reinterpret_cast<Schedule*>(ws + pl.sched);
  int32_t* tok_of_row = reinterpret_cast<int32_t*>(ws + pl.tok_of_row);
  int32_t* row_of_token = reinterpret_cast<int32_t*>(ws + pl.row_of_token);
  rc = routing_launch(role_of_token, head_of_role, n_role, M, T, pl.T_pad, sched, row_of_token,
                      tok_of_row, role_offsets, role_perm, device_status, ws + pl.routing, st);
  if (rc != ATGRPO_OK) return rc;
  LmHeadProblem p;
  p.A_rows = H, p.ldA = ldH, p.rows_bound = T;
  if (M > 1) {
    rc = gather_rows_launch(H, ldH, tok_of_row, pl.T_pad, d, ws + pl.Hs, st);
    if (rc != ATGRPO_OK) return rc;
    p.A_rows = ws + pl.Hs, p.ldA = d, p.rows_bound = pl.T_pad;
  }
  for (int m = 0; m < M; ++m) p.W[m] = W[m];
  p.M = M, p.d = d, p.V = V, p.T = T, p.T_pad = pl.T_pad;
  p.sched = sched, p.tok_of_row = tok_of_row, p.target = target, p.device_status = device_status;
  p.resp_of_token = resp_of_token, p.adv = adv, p.n_resp = n_resp;
  p.n_sm = n_sm;
  rc = lm_head_fwd_launch(p, lse, logp, ws + pl.gemm, st, static_cast<float*>(params->logits), params->logits_format);
  if (rc != ATGRPO_OK) return rc;
  return loss_reduce_launch(logp, old_logp, resp_of_token, adv, n_resp, role_of_token, head_of_role,
                            n_role, M, T, *params, nullptr, loss, nullptr, clip_counts, device_status,
                            ws + pl.loss, st);
}

int atgrpo_policy_loss_bwd(const void* H, int64_t ldH, const void* const* W, int32_t M,
                           const int32_t* target, const int32_t* role_of_token,
                           const int32_t* head_of_role, int32_t n_role,
                           const int32_t* resp_of_token, const float* adv, int64_t n_resp,
                           const float* old_logp, const float* logp, const float* lse,
                           const float* grad_loss, int64_t T, int32_t d, int32_t V,
                           const atgrpo_params* params, void* dH, void* const* dW,
                           int32_t* device_status, void* workspace, size_t workspace_bytes,
                           void* stream) {
  return policy_loss_bwd_impl(H, ldH, W, M, target, role_of_token, head_of_role, n_role, resp_of_token, adv,
                              n_resp, old_logp, logp, lse, grad_loss, T, d, V, params, dH, dW, nullptr, 0,
                              false, device_status, workspace, workspace_bytes, stream);
}

int atgrpo_policy_loss_bwd_chunks(int64_t T, int32_t d, int32_t V, int32_t M, int32_t* n_chunks,
                                  int32_t* rows_per_chunk) {
  if (T < 0 || d < 1 || M < 1 || V < 1 || n_chunks == nullptr || rows_per_chunk == nullptr) return ATGRPO_ERR_INVALID_ARG;
  const int64_t T_pad = padded_rows(T, M);
  *n_chunks = lm_head_bwd_chunks(T_pad, d, V);
  *rows_per_chunk = lm_head_bwd_chunk_rows(T_pad, d, V);
  return ATGRPO_OK;
}

int atgrpo_policy_loss_bwd_notify(const void* H, int64_t ldH, const void* const* W, int32_t M,
                                  const int32_t* target, const int32_t* role_of_token,
                                  const int32_t* head_of_role, int32_t n_role,
                                  const int32_t* resp_of_token, const float* adv, int64_t n_resp,
                                  const float* old_logp, const float* logp, const float* lse,
                                  const float* grad_loss, int64_t T, int32_t d, int32_t V,
                                  const atgrpo_params* params, void* dH, void* const* dW,
                                  void* const* chunk_events, int32_t n_events, int32_t* device_status,
                                  void* workspace, size_t workspace_bytes, void* stream) {
  return policy_loss_bwd_impl(H, ldH, W, M, target, role_of_token, head_of_role, n_role, resp_of_token, adv,
                              n_resp, old_logp, logp, lse, grad_loss, T, d, V, params, dH, dW, chunk_events,
                              n_events, true, device_status, workspace, workspace_bytes, stream);
}

}  // extern "C"

namespace {
int policy_loss_bwd_impl(const void* H, int64_t ldH, const void* const* W, int32_t M,
                         const int32_t* target, const int32_t* role_of_token,
                         const int32_t* head_of_role, int32_t n_role,
                         const int32_t* resp_of_token, const float* adv, int64_t n_resp,
                         const float* old_logp, const float* logp, const float* lse,
                         const float* grad_loss, int64_t T, int32_t d, int32_t V,
                         const atgrpo_params* params, void* dH, void* const* dW,
                         void* const* chunk_events, int32_t n_events, bool notify,
                         int32_t* device_status, void* workspace, size_t workspace_bytes,
                         void* stream) {
  int rc = policy_common_checks(H, ldH, W, M, target, role_of_token, head_of_role, n_role,
                                resp_of_token, adv, n_resp, old_logp, T, d, V, params, workspace);
  if (rc != ATGRPO_OK) return rc;
  if (dW == nullptr) return ATGRPO_ERR_INVALID_ARG;
  if (notify) {
    if (chunk_events == nullptr || n_events != lm_head_bwd_chunks(padded_rows(T, M), d, V)) return ATGRPO_ERR_INVALID_ARG;
    for (int c = 0; c < n_events; ++c)
      if (chunk_events[c] == nullptr) return ATGRPO_ERR_INVALID_ARG;
  }
  for (int m = 0; m < M; ++m)
    if (dW[m] == nullptr || !aligned(dW[m], 32)) return ATGRPO_ERR_INVALID_ARG;
  if (T > 0 && (logp == nullptr || lse == nullptr || dH == nullptr || !aligned(dH, 32)))
    return ATGRPO_ERR_INVALID_ARG;
  int n_sm = 0, cc = 0;
  if (device_sm_count(&n_sm, &cc) != ATGRPO_OK) return ATGRPO_ERR_CUDA;
  if (cc != 10) return ATGRPO_ERR_UNSUPPORTED;
  const PolicyPlan pl = policy_plan(T, d, V, M, true, false, n_sm);
  if (workspace_bytes < pl.total) return ATGRPO_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  const size_t dw_elem = params->dW_dtype == ATGRPO_BF16 ? 2 : 4;
  if (T == 0) {
    if (!params->accumulate_dW)
      for (int m = 0; m < M; ++m)
        ATGRPO_CUDA_OK(cudaMemsetAsync(dW[m], 0, (size_t)V * d * dw_elem, st));
    for (int c = 0; notify && c < n_events; ++c)
      ATGRPO_CUDA_OK(cudaEventRecord(static_cast<cudaEvent_t>(chunk_events[c]), st));
    return ATGRPO_OK;
  }
  Schedule* sched = reinterpret_cast<Schedule*>(ws + pl.sched);
  int32_t* tok_of_row = reinterpret_cast<int32_t*>(ws + pl.tok_of_row);
  int32_t* row_of_token = reinterpret_cast<int32_t*>(ws + pl.row_of_token);
  float* coef = reinterpret_cast<float*>(ws + pl.coef);
  rc = routing_launch(role_of_token, head_of_role, n_role, M, T, pl.T_pad, sched, row_of_token,
                      tok_of_row, nullptr, nullptr, device_status, ws + pl.routing, st);
  if (rc != ATGRPO_OK) return rc;
  if (params->reduction != ATGRPO_REDUCE_TOKEN_MEAN)
    rc = loss_reduce_launch(logp, old_logp, resp_of_token, adv, n_resp, role_of_token, head_of_role,
                            n_role, M, T, *params, grad_loss, nullptr, coef, nullptr, device_status,
                            ws + pl.loss, st);
  else
    rc = coef_launch(logp, old_logp, resp_of_token, adv, n_resp, role_of_token, head_of_role, n_role,
                     M, T, *params, grad_loss, sched, coef, device_status, st);
  if (rc != ATGRPO_OK) return rc;
  // Tokens whose coef is zero (clipped ratio, zero advantage -- e.g. every token of a group whose
  // candidates all got the same reward) contribute exactly nothing to dH and dW: route only the
  // others, so the three backward GEMMs run on the rows that carry a gradient.
  rc = routing_launch(role_of_token, head_of_role, n_role, M, T, pl.T_pad, sched, row_of_token,
                      tok_of_row, nullptr, nullptr, nullptr, ws + pl.routing, st, coef);
  if (rc != ATGRPO_OK) return rc;
  rc = gather_rows_launch(H, ldH, tok_of_row, pl.T_pad, d, ws + pl.Hs, st);
  if (rc != ATGRPO_OK) return rc;
  LmHeadProblem p;
  p.A_rows = ws + pl.Hs, p.ldA = d, p.rows_bound = pl.T_pad;
  for (int m = 0; m < M; ++m) p.W[m] = W[m];
  p.M = M, p.d = d, p.V = V, p.T = T, p.T_pad = pl.T_pad;
  p.sched = sched, p.tok_of_row = tok_of_row, p.target = target, p.device_status = device_status;
  p.resp_of_token = resp_of_token, p.adv = adv, p.n_resp = n_resp;
  p.n_sm = n_sm;
  return lm_head_bwd_launch(p, lse, coef, row_of_token, *params, dH, dW, ws + pl.gemm, st,
                            notify ? chunk_events : nullptr, static_cast<const float*>(params->logits),
                            params->logits_format);
}
}  // namespace

extern "C" {

size_t atgrpo_grad_sumsq_workspace_bytes(void) { return grad_sumsq_workspace_bytes(); }

int atgrpo_grad_sumsq(const void* grad, int32_t grad_dtype, int64_t n, double* sumsq, void* workspace,
                      size_t workspace_bytes, void* stream) {
  if (n < 0 || sumsq == nullptr || (grad_dtype != ATGRPO_F32 && grad_dtype != ATGRPO_BF16))
    return ATGRPO_ERR_INVALID_ARG;
  if (n > 0 && (grad == nullptr || !aligned(grad, 16))) return ATGRPO_ERR_INVALID_ARG;
  if (workspace == nullptr || !aligned(workspace, 256) || workspace_bytes < grad_sumsq_workspace_bytes())
    return ATGRPO_ERR_WORKSPACE;
  return grad_sumsq_launch(grad, grad_dtype, n, sumsq, workspace, static_cast<cudaStream_t>(stream));
}

int atgrpo_adamw_step(const void* grad, int32_t grad_dtype, float* master, float* m, float* v,
                      void* w_bf16, int64_t n, const double* grad_sumsq,
                      const atgrpo_adamw_params* p, void* stream) {
  if (p == nullptr || n < 0 || (grad_dtype != ATGRPO_F32 && grad_dtype != ATGRPO_BF16))
    return ATGRPO_ERR_INVALID_ARG;
  if (p->step < 1 || !(p->beta1 >= 0.f && p->beta1 < 1.f) || !(p->beta2 >= 0.f && p->beta2 < 1.f) ||
      !(p->eps >= 0.f) || !(p->lr >= 0.f) || !(p->weight_decay >= 0.f))
    return ATGRPO_ERR_INVALID_ARG;
  if (n == 0) return ATGRPO_OK;
  if (grad == nullptr || master == nullptr || m == nullptr || v == nullptr) return ATGRPO_ERR_INVALID_ARG;
  if (!aligned(grad, 16) || !aligned(master, 16) || !aligned(m, 16) || !aligned(v, 16) ||
      (w_bf16 != nullptr && !aligned(w_bf16, 16)))
    return ATGRPO_ERR_INVALID_ARG;
  return adamw_launch(grad, grad_dtype, master, m, v, w_bf16, n, grad_sumsq, p->lr, p->beta1, p->beta2,
                      p->eps, p->weight_decay, p->max_grad_norm, p->step, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
