// Internal launch interfaces between the translation units of libatgrpo.
#pragma once
#include "common.cuh"

namespace atgrpo {

// Validation of the scalar parameters, shared by every entry point that takes atgrpo_params.
inline bool params_ok(const atgrpo_params* p) {
  if (p == nullptr) return false;
  if (!(p->clip_eps_low >= 0.f) || !(p->clip_eps_high >= 0.f) || !(p->std_eps >= 0.f)) return false;   // NaN fails too
  if (p->ddof != 0 && p->ddof != 1) return false;
  if (p->dH_dtype != ATGRPO_BF16 && p->dH_dtype != ATGRPO_F32) return false;
  if (p->dW_dtype != ATGRPO_BF16 && p->dW_dtype != ATGRPO_F32) return false;
  if (p->reduction != ATGRPO_REDUCE_TOKEN_MEAN && p->reduction != ATGRPO_REDUCE_SEQUENCE &&
      p->reduction != ATGRPO_REDUCE_GROUP_MEAN)
    return false;
  if (p->candidates_grouped != 0 && p->candidates_grouped != 1) return false;
  if (p->logits_format != ATGRPO_LOGITS_F32 && p->logits_format != ATGRPO_LOGITS_Q16) return false;
  if (p->reduction == ATGRPO_REDUCE_GROUP_MEAN &&
      (p->group_of_resp == nullptr || p->group_scratch == nullptr || p->n_groups < 1))
    return false;
  return true;
}

// ---- group_adv.cu ---------------------------------------------------------------------------
// Optional extras of the advantage pipeline: Eq. 3 reward mix (rewards = alpha*r_team + r_loc,
// written to rewards_out if given) and the per-group argmax candidate (group_best[G], -1 = empty).
// Only with the sort-free pipeline (no bucketing outputs).
struct GroupExtras {
  const float* r_team;
  const float* r_loc;
  float alpha;
  float* rewards_out;
  int32_t* group_best;
};
size_t group_select_workspace_bytes(int64_t n_cand, int64_t n_groups);
size_t group_adv_workspace_bytes(int64_t n_cand, int64_t n_groups);
int group_adv_launch(const float* rewards, const int32_t* env_id, const int32_t* role_id,
                     const int32_t* turn_id, int64_t n_cand, int32_t n_env, int32_t n_role,
                     int32_t n_turn, const atgrpo_params& prm, float* adv, int32_t* group_of_cand,
                     int32_t* group_offsets, int32_t* group_perm, float* group_mean,
                     float* group_std, int32_t* device_status, void* workspace, cudaStream_t st,
                     const GroupExtras* extras = nullptr, bool packed = false);

// Padded 128-row tile schedule the GEMM kernels read.
struct Schedule {                       // lives in device memory
  int32_t n_heads;
  int32_t tile_begin[ATGRPO_MAX_HEADS + 1];   // first 128-row tile of head m in the padded row space
  int32_t rows[ATGRPO_MAX_HEADS];             // T_m
  int32_t role_offsets[ATGRPO_MAX_HEADS + 1]; // exclusive scan of T_m
};

// ---- loss_reduce.cu -------------------------------------------------------------------------
// Eq. 2 reduction for up to ATGRPO_MAX_HEADS policies: token mean (coef only for M == 1) or,
// with prm.reduction == ATGRPO_REDUCE_SEQUENCE / _GROUP_MEAN, per-response ratios and the mean
// over responses / over groups of the per-group mean (coef for any M, scaled by grad_loss[m] / R_m
// or grad_loss[m] / (K_g G_m); loss may be NULL).
size_t loss_reduce_workspace_bytes(int64_t T);
int loss_reduce_launch(const float* logp, const float* old_logp, const int32_t* resp_of_token,
                       const float* adv, int64_t n_resp, const int32_t* role_of_token,
                       const int32_t* head_of_role, int32_t n_role, int32_t M, int64_t T,
                       const atgrpo_params& prm, const float* grad_loss, float* loss, float* coef,
                       int64_t* clip_counts, int32_t* device_status, void* workspace, cudaStream_t st);

// coef[j] = grad_loss[m]*A*rho*[gradient passes]/T_m for every token (0 where unroutable).
int coef_launch(const float* logp, const float* old_logp, const int32_t* resp_of_token,
                const float* adv, int64_t n_resp, const int32_t* role_of_token,
                const int32_t* head_of_role, int32_t n_role, int32_t M, int64_t T,
                const atgrpo_params& prm, const float* grad_loss, const Schedule* sched,
                float* coef, int32_t* device_status, cudaStream_t st);

// Stable routing of tokens to heads plus the padded 128-row tile schedule the GEMM kernels read.
size_t routing_workspace_bytes(int64_t T, int32_t M);
// Writes sched, row_of_token[T] (padded row of each token, -1 if unroutable) and tok_of_row[T_pad]
// (-1 for padding rows); optional role_offsets / role_perm outputs.  With keep_if_nonzero[T] only
// the tokens with a non-zero entry are routed (the others get row -1).
int routing_launch(const int32_t* role_of_token, const int32_t* head_of_role, int32_t n_role,
                   int32_t M, int64_t T, int64_t T_pad, Schedule* sched, int32_t* row_of_token,
                   int32_t* tok_of_row, int32_t* role_offsets, int32_t* role_perm,
                   int32_t* device_status, void* workspace, cudaStream_t st,
                   const float* keep_if_nonzero = nullptr);
// Hs[row] = H[tok_of_row[row]] (zeros for padding rows); rows of d bf16, 16-byte vectors.
int gather_rows_launch(const void* H, int64_t ldH, const int32_t* tok_of_row, int64_t T_pad,
                       int32_t d, void* Hs, cudaStream_t st);

// ---- optimizer.cu ---------------------------------------------------------------------------
size_t grad_sumsq_workspace_bytes();
int grad_sumsq_launch(const void* grad, int grad_dtype, int64_t n, double* sumsq_out, void* workspace,
                      cudaStream_t st);
int adamw_launch(const void* grad, int grad_dtype, float* master, float* m, float* v, void* w_bf16,
                 int64_t n, const double* sumsq, float lr, float beta1, float beta2, float eps,
                 float weight_decay, float max_norm, int step, cudaStream_t st);

// ---- lm_head.cu -----------------------------------------------------------------------------
struct LmHeadProblem {
  const void* A_rows;        // bf16 [rows_total, d] rows in padded order (H itself when M == 1)
  int64_t ldA;               // row stride of A_rows in elements
  int64_t rows_bound;        // rows addressable through A_rows (T when M == 1, T_pad otherwise)
  const void* W[ATGRPO_MAX_HEADS];
  int32_t M, d, V;
  int64_t T, T_pad;
  const Schedule* sched;     // device
  const int32_t* tok_of_row; // device, [T_pad]
  const int32_t* target;     // device, [T] in token order
  const int32_t* resp_of_token;   // device, [T]; with adv[n_resp]: read by the forward only when it keeps the logits
  const float* adv;
  int64_t n_resp;
  int32_t* device_status;
  int32_t n_sm;
};
size_t lm_head_fwd_workspace_bytes(int64_t T_pad, int32_t d, int32_t V, int32_t n_sm);
// lse[T], logp[T] in token order.  keep_logits (optional): lm_head_logits_bytes(T, V, logits_format)
// bytes; receives the logits of every routed token that can carry a gradient, rows in token order with
// stride lm_head_logits_ld(V): fp32, or 16-bit codes followed by one fp32 per 32-column block.
int64_t lm_head_logits_ld(int32_t V);
size_t lm_head_logits_bytes(int64_t T, int32_t V, int32_t format);
int lm_head_fwd_launch(const LmHeadProblem& p, float* lse, float* logp, void* workspace,
                       cudaStream_t st, float* keep_logits = nullptr, int32_t logits_format = ATGRPO_LOGITS_F32);
size_t lm_head_bwd_workspace_bytes(int64_t T_pad, int32_t d, int32_t V, bool dH_direct);
// coef[T] in token order (0 for tokens that pass no gradient); dH / dW as the C ABI documents.
// chunk_events (optional, lm_head_bwd_chunks() entries): event c is recorded once the dW rows of
// vocabulary chunk c are final.  kept_logits (optional): what the forward call stored through
// keep_logits for the same H, W and routing inputs; dZ is then formed from it instead of a second contraction.
int lm_head_bwd_launch(const LmHeadProblem& p, const float* lse, const float* coef,
                       const int32_t* row_of_token, const atgrpo_params& prm, void* dH,
                       void* const* dW, void* workspace, cudaStream_t st,
                       void* const* chunk_events = nullptr, const float* kept_logits = nullptr,
                       int32_t logits_format = ATGRPO_LOGITS_F32);
int lm_head_bwd_chunk_rows(int64_t T_pad, int32_t d, int32_t V);   // vocabulary rows per chunk
int device_sm_count(int* n_sm, int* cc_major);
int lm_head_bwd_chunks(int64_t T_pad, int32_t d, int32_t V);   // vocabulary chunks of one backward call (it makes one GEMM launch more)

}  // namespace atgrpo
