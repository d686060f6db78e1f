/*
 * atgrpo.h -- C ABI of libatgrpo: the data-parallel hot path of the AT-GRPO policy update
 * (arXiv 2510.11062) for NVIDIA B200 (sm_100a).
 *
 * Two operations of the paper are exported:
 *   - the agent- and turn-wise group-relative advantage (Eq. 1 applied to the groups that the
 *     group-key step of Algorithm 1 forms, one per environment, agent and turn), and
 *   - the clipped-ratio policy loss (Eq. 2) through the LM head, forward and backward, for one
 *     shared policy (M = 1) or one policy per role (M = N), Sec. 3 "Role-sharing vs.
 *     Role-specialized Policy Optimization".
 *
 * Conventions common to every entry point
 *   - Every pointer is a DEVICE pointer owned by the caller unless its comment says "host".
 *     The library allocates no memory, never synchronises the device and enqueues all work on
 *     `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream).  It keeps no
 *     state between calls apart from two host-side lookups made once per process and cached: the
 *     driver entry point that encodes tensor maps, and (atgrpo_group_advantages_noalloc only) the
 *     device address of its built-in scratch array, per device.  Scratch comes from `workspace`, at least as many bytes as the
 *     matching *_workspace_bytes() query returns, 256-byte aligned, private to the call
 *     until the enqueued work has finished.
 *   - Return value: ATGRPO_OK, or an error detected on the host, in which case nothing was
 *     enqueued and no output was touched.
 *   - Problems only the device can see (an index outside its range, a bounded wait that ran
 *     out) are reported through `device_status`, one int32 in device memory that the caller
 *     zeroes: the first error code is written there (first writer wins, later ones keep it),
 *     the offending element is skipped without any out-of-bounds access and the kernels run to
 *     completion.  No entry point traps, asserts or aborts.
 *   - Arrays are dense and row-major.  int32 index arrays, fp32 statistics, bf16 operands.
 *   - Calls may run concurrently on different streams if they use different workspaces and
 *     different outputs.
 */
#ifndef ATGRPO_H_
#define ATGRPO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum atgrpo_status {
  ATGRPO_OK = 0,
  ATGRPO_ERR_INVALID_ARG = 1, /* NULL where data is required, negative size, bad enum       */
  ATGRPO_ERR_UNSUPPORTED = 2, /* device is not sm_100, d not a multiple of 8, M too large ... */
  ATGRPO_ERR_WORKSPACE = 3,   /* workspace NULL, misaligned or too small                      */
  ATGRPO_ERR_BAD_INDEX = 4,   /* device-detected: an id / token / role outside its range      */
  ATGRPO_ERR_TIMEOUT = 5,     /* device-detected: a bounded wait inside a kernel expired      */
  ATGRPO_ERR_CUDA = 6,        /* a CUDA runtime or driver call failed on the host             */
  ATGRPO_ERR_LAYOUT = 7       /* device-detected: params->candidates_grouped was set, but the  */
                              /* members of some group are not adjacent                       */
} atgrpo_status;

enum { ATGRPO_BF16 = 0, ATGRPO_F32 = 1 };

/* Largest number of policies (LM heads) one call can route to. */
#define ATGRPO_MAX_HEADS 8

/* Scalars of Eq. 1 and Eq. 2.  The paper gives the symbols, not the values: epsilon of Eq. 2 is
 * clip_eps_low / clip_eps_high (0.2 both in all shipped workloads); F_norm of Eq. 1 is
 * std + std_eps with the population (ddof = 0) or Bessel (ddof = 1) standard deviation. */
typedef struct atgrpo_params {
  float clip_eps_low;
  float clip_eps_high;
  float std_eps;
  int32_t ddof;
  int32_t dH_dtype;      /* ATGRPO_BF16 (default) or ATGRPO_F32: element type of dH            */
  int32_t dW_dtype;      /* ATGRPO_F32 (default) or ATGRPO_BF16: element type of every dW_m    */
  int32_t accumulate_dW; /* 0: dW_m is overwritten; 1: dW_m += gradient (gradient accumulation)*/
  int32_t reduction;     /* ATGRPO_REDUCE_TOKEN_MEAN (default), _SEQUENCE or _GROUP_MEAN           */
  int32_t candidates_grouped; /* atgrpo_group_advantages only.  0 (default): candidates in any order.
                               * 1: the caller promises that the members of every group are adjacent,
                               * the order Algorithm 1 appends them in (the K samples of one
                               * (environment, agent, turn) together); groups may follow one another
                               * in any order.  The advantages are then computed in one streaming
                               * pass.  The promise is checked on the device: a group that shows up in
                               * two places raises ATGRPO_ERR_LAYOUT, and its members get the statistics
                               * of their own stretch.  Ignored when bucketing outputs are requested. */
  /* ATGRPO_REDUCE_GROUP_MEAN only (ignored otherwise; NULL / 0 by default): */
  const int32_t* group_of_resp; /* device, [n_resp]: group g of every response, in [0, n_groups)
                                 * (what atgrpo_group_advantages writes to group_of_cand)        */
  int32_t* group_scratch;       /* device, [n_groups] int32 owned by the caller, private to the call
                                 * while it runs; the library zeroes it and counts K_g in it      */
  int32_t n_groups;
  /* atgrpo_policy_loss_fwd / _bwd / _bwd_notify only (NULL / 0 by default): logits kept from the
   * forward call for the backward call, see atgrpo_policy_loss_logits_bytes().                  */
  void* logits;                 /* device, 256-byte aligned, owned by the caller                    */
  size_t logits_bytes;          /* size of that buffer in bytes                                     */
  int32_t logits_format;        /* ATGRPO_LOGITS_F32 (default) or ATGRPO_LOGITS_Q16                 */
} atgrpo_params;

/* Readings of the expectation in Eq. 2.
 * TOKEN_MEAN: one ratio per response token, loss_m = mean over all response tokens of policy m.
 * SEQUENCE  : Eq. 2 as printed -- one ratio per response, r_c = pi(o_c|q)/pi_old(o_c|q) =
 *             exp(sum of logp - old_logp over the response's tokens), loss_m = mean over the
 *             responses of policy m that have tokens; every token of response c then carries
 *             coef = grad_loss[m]*A_c*r_c*[unclipped branch active]/R_m.  Requires the tokens packed
 *             response by response (resp_of_token non-decreasing; a violation raises
 *             ATGRPO_ERR_BAD_INDEX); clip counts are per response.
 * GROUP_MEAN: the expectation of Eq. 2 exactly as printed, E_g[(1/K) sum_c .]: sequence-level
 *             ratios as above, loss_m = mean over the groups g of policy m of the mean over the
 *             K_g responses of g that have tokens, so every group weighs the same however many
 *             candidates it kept (K varies when rollouts end early).  Token j of response c in
 *             group g carries coef = grad_loss[m]*A_c*r_c*[active]/(K_g*G_m), G_m = groups of
 *             policy m with at least one such response.  Needs params->group_of_resp,
 *             group_scratch and n_groups; all responses of a group must belong to one policy.
 *             A group id out of range raises ATGRPO_ERR_BAD_INDEX and the response is left out. */
enum { ATGRPO_REDUCE_TOKEN_MEAN = 0, ATGRPO_REDUCE_SEQUENCE = 1, ATGRPO_REDUCE_GROUP_MEAN = 2 };

/* Text for a status code (static storage, never NULL). */
const char* atgrpo_status_string(int status);

/* ------------------------------------------------------------------------------------------
 * Grouped advantage -- Eq. 1 over the (environment, agent, turn) groups of Algorithm 1.
 *
 * Candidate c (one sampled response) carries reward rewards[c] and the ids env_id[c] in
 * [0,n_env), role_id[c] in [0,n_role), turn_id[c] in [0,n_turn); candidates may come in any
 * order.  Its group is g = (env*n_role + role)*n_turn + turn, a collision-free stand-in for the
 * paper's hash(e,i,t); G = n_env*n_role*n_turn slots, empty slots allowed, G < 2^31.
 * For each non-empty group of K members: mu = mean, sigma = std (params->ddof), and
 *   adv[c] = (rewards[c] - mu) / (sigma + params->std_eps);   K = 1 gives adv = 0.
 * The result is bit-reproducible and a group of identical rewards yields exact zeros (sums in
 * ascending candidate order when bucketing outputs are requested or candidates_grouped is set --
 * fp64, or, for adjacent groups of up to 16 members, fp32 on rewards shifted by the group's first
 * one; exact integer accumulation of rewards quantised to 2^-25 of the group's range otherwise).
 *
 * Outputs: adv[n_cand] (required).  Optional (NULL to skip): group_of_cand[n_cand] = g;
 * group_offsets[G+1] and group_perm[n_cand], the stable bucketing (slot s owns
 * group_perm[group_offsets[s] .. group_offsets[s+1]) in ascending candidate index);
 * group_mean[G], group_std[G] (0 for empty slots).
 * A candidate with an id out of range raises ATGRPO_ERR_BAD_INDEX in *device_status, gets
 * adv = 0 and belongs to no group.
 * n_cand = 0 is valid (offsets are zero-filled).  n_cand < 2^31.
 * ------------------------------------------------------------------------------------------ */
size_t atgrpo_group_advantages_workspace_bytes(int64_t n_cand, int64_t n_groups);

int atgrpo_group_advantages(
    const float* rewards, const int32_t* env_id, const int32_t* role_id, const int32_t* turn_id,
    int64_t n_cand, int32_t n_env, int32_t n_role, int32_t n_turn,
    const atgrpo_params* params /* host */,
    float* adv,
    int32_t* group_of_cand, int32_t* group_offsets, int32_t* group_perm,
    float* group_mean, float* group_std,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Grouped advantage from ready-made group ids -- Eq. 1 again, for callers that already hold the
 * group key of Algorithm 1 as one dense id per candidate (for instance the group_of_cand output
 * of an earlier call, or an id assigned when the rollout was stored under its key): group_id[c]
 * in [0, n_groups) replaces the three id arrays, which saves 8 of the 20 bytes the call moves per
 * candidate.  Everything else -- params (ddof, std_eps, candidates_grouped), outputs, error
 * reporting (an id out of range raises ATGRPO_ERR_BAD_INDEX and gets adv = 0), workspace size
 * (atgrpo_group_advantages_workspace_bytes) -- is as in atgrpo_group_advantages.
 * ------------------------------------------------------------------------------------------ */
int atgrpo_group_advantages_packed(
    const float* rewards, const int32_t* group_id, int64_t n_cand, int64_t n_groups,
    const atgrpo_params* params /* host */,
    float* adv,
    int32_t* group_offsets, int32_t* group_perm,
    float* group_mean, float* group_std,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Credit assignment, advantage and greedy selection in one call -- Eq. 3, Eq. 1 and the greedy
 * selection step of Algorithm 1's tree-structured sampling (the best candidate of a group).
 *
 * rewards[c] = alpha*r_team[c] + r_loc[c] (Eq. 3, one fused multiply-add, fp32); advantages as in
 * atgrpo_group_advantages over these rewards; group_best[g] = the candidate of group g with the
 * highest reward (ties: lowest candidate index; -1 for an empty slot), i.e. the action that
 * continues the rollout.  Optional outputs (NULL to skip): rewards_out[n_cand], group_best[G],
 * group_of_cand, group_mean, group_std.  No bucketing outputs here (use atgrpo_group_advantages).
 * ------------------------------------------------------------------------------------------ */
size_t atgrpo_group_select_workspace_bytes(int64_t n_cand, int64_t n_groups);

int atgrpo_group_select(
    const float* r_team, const float* r_loc, float alpha,
    const int32_t* env_id, const int32_t* role_id, const int32_t* turn_id,
    int64_t n_cand, int32_t n_env, int32_t n_role, int32_t n_turn,
    const atgrpo_params* params /* host */,
    float* rewards_out, float* adv, int32_t* group_best,
    int32_t* group_of_cand, float* group_mean, float* group_std,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Grouped advantage without a workspace.  The paper has no counterpart to this entry point; it
 * exists for callers that must not allocate device memory where the advantages are computed:
 * a process that shares the GPU with an inference engine under a fixed memory budget, a plugin
 * whose host application owns every allocation, or a training loop whose caching allocator must
 * not be disturbed between steps.  Same arguments, results and error reporting as
 * atgrpo_group_advantages, minus `workspace`: the scratch is a fixed 4 MiB array inside the
 * library's device image (held by every GPU that loads the library until the process exits).
 * Limits: n_cand <= ATGRPO_NOALLOC_MAX_CAND and n_env*n_role*n_turn <= ATGRPO_NOALLOC_MAX_GROUPS;
 * anything larger returns ATGRPO_ERR_UNSUPPORTED with nothing enqueued.
 * The call makes no cudaMalloc / cudaFree and calls no allocating routine.  The first call on a
 * device looks up the array's device address (cudaGetSymbolAddress, with that device current)
 * and remembers it for the life of the process (the remembered address does not survive a
 * cudaDeviceReset); make that first call before starting any stream capture.
 * All calls on one device share the one array, which keeps the previous call's contents; each
 * call clears what it needs to start from zero.  Two calls whose kernels can overlap on the GPU
 * (different streams without an ordering between them) race on the array: serialise them.
 * ------------------------------------------------------------------------------------------ */
#define ATGRPO_NOALLOC_MAX_CAND 262144
#define ATGRPO_NOALLOC_MAX_GROUPS 65536

int atgrpo_group_advantages_noalloc(
    const float* rewards, const int32_t* env_id, const int32_t* role_id, const int32_t* turn_id,
    int64_t n_cand, int32_t n_env, int32_t n_role, int32_t n_turn,
    const atgrpo_params* params /* host */,
    float* adv,
    int32_t* group_of_cand, int32_t* group_offsets, int32_t* group_perm,
    float* group_mean, float* group_std,
    int32_t* device_status, void* stream);

/* ------------------------------------------------------------------------------------------
 * Clipped-ratio loss from given log-probabilities -- Eq. 2 alone, one policy.
 *
 * For response token j: rho = exp(logp[j] - old_logp[j]), A = adv[resp_of_token[j]]
 * (token-level credit: every response token carries its response's advantage, Sec. 4.1),
 *   l_j = -min(rho*A, clip(rho, 1-eps_low, 1+eps_high)*A),   loss[0] = (1/T) sum_j l_j,
 * summed in fp64 in a fixed order (bit-reproducible).  T = 0 gives loss = 0.
 * Optional outputs: coef[T] = A*rho*[unclipped branch active]/T, the factor of
 * d loss / d logit_jv = coef_j*(p_jv - [v = y_j]); clip_counts[2] (int64) = number of tokens with
 * rho < 1-eps_low and with rho > 1+eps_high.
 * resp_of_token[j] outside [0,n_resp) raises ATGRPO_ERR_BAD_INDEX; the token counts with A = 0.
 * ------------------------------------------------------------------------------------------ */
size_t atgrpo_clipped_loss_workspace_bytes(int64_t T);

int atgrpo_clipped_loss(
    const float* logp, const float* old_logp, const int32_t* resp_of_token, const float* adv,
    int64_t T, int64_t n_resp, const atgrpo_params* params /* host */,
    float* loss, float* coef, int64_t* clip_counts,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Policy loss through the LM head, forward -- Eq. 2 with pi_theta evaluated by the head.
 *
 * H[T, d] (bf16, row stride ldH elements, ldH >= d, ldH % 8 == 0, 16-byte aligned base) holds,
 * for every packed response token j, the hidden state that predicts it.  W is a HOST array of
 * M device pointers, W[m] = bf16 [V, d] contiguous (16-byte aligned): the head of policy m.
 * target[j] in [0,V) is the sampled token.  Policy of token j: m = head_of_role[role_of_token[j]]
 * (sigma of the paper) when M > 1; with M == 1 both arrays may be NULL and every token uses W[0].
 *   z_jv = <H_j, W_m[v]>  (bf16 x bf16, fp32 accumulation on tensor cores; stored only if
 *                          params->logits is given)
 *   lse[j]  = log sum_v exp(z_jv)          logp[j] = z_{j,target[j]} - lse[j]
 *   rho_j = exp(logp[j] - old_logp[j]),  A = adv[resp_of_token[j]]
 *   loss[m] = (1/T_m) sum_{j of policy m} -min(rho_j*A, clip(rho_j)*A)   (0 if T_m = 0)
 * Outputs: loss[M], logp[T], lse[T] (lse and logp are what the backward call needs).
 * Optional: role_offsets[M+1], role_perm[T] = stable routing of tokens to policies (tokens of
 * policy m in ascending token index); clip_counts[M*2] (int64) as in atgrpo_clipped_loss.
 * Requirements: d % 8 == 0, d >= 64, V >= 1, 1 <= M <= ATGRPO_MAX_HEADS, T < 2^31 - 2^16.
 * Out-of-range indices raise ATGRPO_ERR_BAD_INDEX in *device_status and stay in bounds: a bad
 * target is read as token 0; a token whose role or head is out of range belongs to no policy
 * (its logp and lse are left untouched, it enters no loss); a bad response index counts the
 * token with A = 0.
 * ------------------------------------------------------------------------------------------ */
size_t atgrpo_policy_loss_workspace_bytes(int64_t T, int32_t d, int32_t V, int32_t M, int32_t is_bwd);

/* Kept logits (optional; a memory / compute trade the paper says nothing about).  The gradient of
 * Eq. 2 needs the softmax pi_theta(v | .) of every token that passes a gradient, i.e. its logits
 * again.  By default the backward call repeats the contraction z = H W_m^T chunk by chunk
 * (2*T*V*d flop more, no memory).  A caller with HBM to spare can instead lend params->logits, a
 * buffer of atgrpo_policy_loss_logits_bytes(T, V, ATGRPO_LOGITS_F32) bytes = T rows of V rounded
 * up to a multiple of 256 fp32 values (9.8 GB at T = 16157, V = 151936): the forward call then also stores
 * z_jv (row j = token j, columns >= V unspecified; rows of tokens that belong to no policy, or
 * whose response has advantage 0 and therefore passes no gradient, are left untouched), and a
 * backward call that is given the same buffer -- after a forward call
 * with the same H, W, target, adv and routing arguments, nothing having written to it in between --
 * reads the logits back instead of recomputing them: a quarter less tensor work for one write and
 * one read of the buffer.  With fp32 logits both ways produce bit-identical dH and dW.  A buffer that is
 * misaligned or too small is rejected with ATGRPO_ERR_INVALID_ARG; the library cannot tell
 * whether the contents belong to these inputs.
 * params->logits_format = ATGRPO_LOGITS_Q16 halves the buffer and its traffic (2.125 bytes per logit):
 * the buffer then holds, for every token, V rounded up to a multiple of 256 uint16 codes and, after
 * the codes of all tokens, one fp32 per token and 32-column block (the block's largest logit);
 * z_jv is stored as q = round((max of its block - z_jv) * 1024), clamped at 65535, and read back as
 * max - q/1024: |error| <= 2^-11 for every logit within 64 of its block's maximum (anything lower
 * is read as max - 64, where exp(z - lse) is below 2e-28 of the block's largest softmax value), i.e.
 * at most 4.9e-4 relative on every softmax value, a quarter of what rounding dZ to bf16 contributes.
 * dH and dW then stay within the stated tolerances but are no longer bit-identical to the
 * recomputing call; logits that are not finite are not preserved by this format. */
enum { ATGRPO_LOGITS_F32 = 0, ATGRPO_LOGITS_Q16 = 1 };
size_t atgrpo_policy_loss_logits_bytes(int64_t T, int32_t V, int32_t logits_format);

/* Number of kernels one forward (is_bwd = 0) or backward (is_bwd = 1) call enqueues for these
 * sizes on the current device (memsets not counted).  A bookkeeping query with no counterpart in
 * the paper: callers use it to size CUDA graphs and to report launch counts. */
int32_t atgrpo_policy_loss_launch_count(int64_t T, int32_t d, int32_t V, int32_t M, int32_t is_bwd);

int atgrpo_policy_loss_fwd(
    const void* H, int64_t ldH, const void* const* W /* host array */, int32_t M,
    const int32_t* target,
    const int32_t* role_of_token, const int32_t* head_of_role, int32_t n_role,
    const int32_t* resp_of_token, const float* adv, int64_t n_resp,
    const float* old_logp,
    int64_t T, int32_t d, int32_t V, const atgrpo_params* params /* host */,
    float* loss, float* logp, float* lse,
    int32_t* role_offsets, int32_t* role_perm, int64_t* clip_counts,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Policy loss through the LM head, backward -- gradient of sum_m grad_loss[m]*loss[m] (Eq. 2)
 * with respect to H and every W_m (the update theta_m <- theta_m - eta*grad L of Sec. 3).
 *
 * Inputs as in the forward call, plus logp[T] and lse[T] as the forward call wrote them and
 * grad_loss[M] (device; NULL = all ones).  With
 *   coef_j = grad_loss[m]*A*rho_j*[rho_j*A <= clip(rho_j)*A and A != 0]/T_m,
 * the softmax is recomputed tile by tile, p_jv = exp(z_jv - lse[j]), and
 *   dZ_jv = coef_j*(p_jv - [v = target[j]])   (rounded to bf16 for the contractions)
 *   dH[j, :]   = sum_v dZ_jv * W_m[v, :]          -> dH [T, d], row stride d, params->dH_dtype
 *   dW[m][v,:] = sum_{j of policy m} dZ_jv*H[j,:] -> dW[m] [V, d] contiguous, params->dW_dtype,
 *                overwritten or accumulated into (params->accumulate_dW).
 * dW is a HOST array of M device pointers; dH and every dW[m] must be 32-byte aligned.
 * A policy without tokens gets dW = 0 (or is left unchanged when accumulating).  The [T, V]
 * gradient of the logits is never materialised: dZ lives in a bounded vocabulary-chunk buffer
 * inside the workspace; the logits themselves exist in memory only if the caller lends
 * params->logits (then they are read from there instead of being recomputed).
 * ------------------------------------------------------------------------------------------ */
int atgrpo_policy_loss_bwd(
    const void* H, int64_t ldH, const void* const* W /* host array */, int32_t M,
    const int32_t* target,
    const int32_t* role_of_token, const int32_t* head_of_role, int32_t n_role,
    const int32_t* resp_of_token, const float* adv, int64_t n_resp,
    const float* old_logp, const float* logp, const float* lse, const float* grad_loss,
    int64_t T, int32_t d, int32_t V, const atgrpo_params* params /* host */,
    void* dH, void* const* dW /* host array */,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * The backward call with a notification per vocabulary chunk, for data-parallel training: the
 * update of Sec. 3 uses the gradient of the whole batch B_m, so ranks that hold different
 * environments sum their dW_m, and that sum can start on the rows that are final while the rest
 * is still being computed.
 *
 * atgrpo_policy_loss_bwd_chunks: the backward call walks the vocabulary in *n_chunks pieces of
 * *rows_per_chunk rows (the last one shorter); a function of (T, d, V, M) only.
 * atgrpo_policy_loss_bwd_notify: as atgrpo_policy_loss_bwd; in addition chunk_events is a HOST
 * array of n_events CUDA events (cudaEvent_t, created by the caller; n_events must equal
 * n_chunks), and event c is recorded on `stream` as soon as the rows
 * [c*rows_per_chunk, min(V, (c+1)*rows_per_chunk)) of every dW_m are final.  dH is final when the
 * call's last kernel has run, as usual.  With T = 0 all events are recorded after the zero fill.
 * ------------------------------------------------------------------------------------------ */
int atgrpo_policy_loss_bwd_chunks(int64_t T, int32_t d, int32_t V, int32_t M, int32_t* n_chunks,
                                  int32_t* rows_per_chunk);

int atgrpo_policy_loss_bwd_notify(
    const void* H, int64_t ldH, const void* const* W /* host array */, int32_t M,
    const int32_t* target,
    const int32_t* role_of_token, const int32_t* head_of_role, int32_t n_role,
    const int32_t* resp_of_token, const float* adv, int64_t n_resp,
    const float* old_logp, const float* logp, const float* lse, const float* grad_loss,
    int64_t T, int32_t d, int32_t V, const atgrpo_params* params /* host */,
    void* dH, void* const* dW /* host array */,
    void* const* chunk_events /* host array of cudaEvent_t */, int32_t n_events,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Parameter update of one policy's LM head -- theta_m <- theta_m - eta * grad L(theta_m) (Sec. 3)
 * with the optimiser settings of App. "Training Details": gradient clipping at a global L2 norm,
 * Adam with weight decay (read as AdamW: decoupled decay, bias-corrected moments).
 *
 * atgrpo_grad_sumsq: sumsq[0] = sum of squares of the n gradient elements (fp64, device), summed
 * in a fixed order.  The caller may add the squared norm of the policy's other parameters (the
 * transformer trunk is not in this library) before passing it on.
 *
 * atgrpo_adamw_step, for step number `step` >= 1, per element:
 *   g = grad * min(1, max_grad_norm / (sqrt(*grad_sumsq) + 1e-6))    (no clipping if grad_sumsq is
 *                                                                      NULL or max_grad_norm <= 0)
 *   m = beta1*m + (1-beta1)*g          v = beta2*v + (1-beta2)*g*g
 *   master = master*(1 - lr*weight_decay) - lr*(m/(1-beta1^step)) / (sqrt(v/(1-beta2^step)) + eps)
 *   w_bf16 = bf16(master)              (optional output, NULL to skip: the head the loss kernels read)
 * grad has grad_dtype (ATGRPO_F32 or ATGRPO_BF16); master, m, v are fp32 and updated in place.
 * All arrays hold n elements and are 16-byte aligned.  fp32 arithmetic.
 * ------------------------------------------------------------------------------------------ */
typedef struct atgrpo_adamw_params {
  float lr;            /* 1e-6 in the paper */
  float beta1, beta2;  /* not given in the paper; 0.9, 0.999 are the usual defaults */
  float eps;           /* 1e-8 */
  float weight_decay;  /* 0.01 in the paper */
  float max_grad_norm; /* 1.0 in the paper */
  int32_t step;        /* 1-based step count */
} atgrpo_adamw_params;

size_t atgrpo_grad_sumsq_workspace_bytes(void);

int atgrpo_grad_sumsq(const void* grad, int32_t grad_dtype, int64_t n, double* sumsq,
                      void* workspace, size_t workspace_bytes, void* stream);

int atgrpo_adamw_step(const void* grad, int32_t grad_dtype, float* master, float* m, float* v,
                      void* w_bf16, int64_t n, const double* grad_sumsq,
                      const atgrpo_adamw_params* params /* host */, void* stream);

/* ------------------------------------------------------------------------------------------
 * Self-test of the bounded waits (no counterpart in the paper; it exercises the error convention
 * stated at the top of this file).  Every barrier wait inside the LM-head kernels gives up after
 * a wall-clock limit and reports ATGRPO_ERR_TIMEOUT; a healthy run never gets there.  This call
 * enqueues one tiny kernel (one block, no tensor-core or bulk-copy work) whose two waiting warps
 * wait on a barrier that nothing arrives on, with a limit of limit_ns nanoseconds (1 us .. 50 ms),
 * and then return normally.  Afterwards *device_status holds ATGRPO_ERR_TIMEOUT (if it was 0
 * before) and, if `waited` (device, 2 x int32, optional) is given, waited[i] = 1 for each warp
 * whose wait returned "gave up".  The context stays usable: nothing traps or faults.
 * ------------------------------------------------------------------------------------------ */
int atgrpo_selftest_bounded_wait(int64_t limit_ns, int32_t* device_status, int32_t* waited, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ATGRPO_H_ */
