"""Plain fp64 CPU oracle for the AT-GRPO policy-update hot path.

TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
what the CUDA library computes.  It shares no code with the CUDA path and must
never be imported by the product package; only the tests, the smoke check and
the benchmark's CPU-baseline leg call it.

Everything is NumPy in float64.  Each function restates one definition of the
paper (arXiv 2510.11062) in the paper's order and notation:

  group_key            Algorithm 1, group-key step: one key per (environment, agent, turn)
  bucket_by_key        Algorithm 1 / Sec. 4.1 "Agent- and Turn-wise Grouping"
  group_advantages     Eq. 1 (group-relative advantage)
  mix_rewards          Eq. 3 (agent-wise credit assignment: team + local reward)
  group_argmax         Algorithm 1, greedy selection step of the tree-structured sampling
  route_tokens         Sec. 3 "Role-sharing vs. Role-specialized", B_m = U_{sigma(i)=m} D_i
  token_logprobs       pi_theta in Eq. 2: log-softmax of the LM-head logits at the sampled token
  clipped_objective    Eq. 2, per token (token-level credit, Sec. 4.1 "Reward Mask")
  policy_loss          Eq. 2, one loss per policy m (token-level reading)
  policy_loss_sequence Eq. 2 as printed: one ratio per response; mean over the responses of B_m, or
                       (group_of_resp given) mean over groups of the per-group mean over K candidates
  policy_loss_grads    gradient of Eq. 2 w.r.t. the hidden states H and the head W_m
  grad_sumsq, clip_scale, adamw_step
                       the update theta_m <- theta_m - eta*grad L of Sec. 3 with the optimiser
                       settings of App. "Training Details" (Adam, weight decay, gradient clipping)

Readings taken where the paper is silent (each is pinned by a test, none by the
paper's own numbers -- the paper prints no worked example):
  * F_norm of Eq. 1 is the standard deviation of the group's rewards;
    population (ddof=0) by default, Bessel (ddof=1) on request.
  * A = (R - mean) / (std + eps), eps added outside the square root.
  * a group of one candidate has A = 0 (no comparison, no learning signal).
  * the ratio of Eq. 2 is taken per response token and the expectation is the
    mean over all response tokens of policy m's batch.
  * hash(e, i, t) is the collision-free mixed-radix index (e*N + i)*T + t.
  * no KL, entropy or temperature term (entropy coefficient 0, T_sample 1).
  * "Adam ... weight decay 0.01 ... gradient clipping at 1.0" is read as AdamW (decoupled decay,
    Loshchilov & Hutter) with bias correction, after scaling the gradient by
    min(1, max_norm / (global L2 norm + 1e-6)).
Parity status: every function below is pinned by tests/test_oracle_pins.py
against closed forms, invariants, brute force, finite differences or an
independent library routine.  The *readings* above (std convention, eps
placement, token- vs sequence-level ratio, denominator) are "parity unpinned"
by the paper itself.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "group_key", "bucket_by_key", "group_advantages", "mix_rewards", "group_argmax", "route_tokens",
    "token_logprobs", "clipped_objective", "policy_loss", "dloss_dlogp", "policy_loss_grads",
    "policy_loss_sequence", "dloss_dlogp_sequence",
    "policy_loss_grad_rows", "grad_sumsq", "clip_scale", "adamw_step",
]


def _f64(x):
    """Widen any array-like (NumPy array or CPU torch tensor, bf16 included) to float64."""
    if hasattr(x, "detach"):                      # torch tensor, without importing torch here
        x = x.detach().cpu().double().numpy()
    return np.asarray(x, dtype=np.float64)


def _i64(x):
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.asarray(x, dtype=np.int64)


# --------------------------------------------------------------------------- grouping
def group_key(env_id, role_id, turn_id, n_env, n_role, n_turn):
    """Group key of Algorithm 1: one key per (environment e, agent i, turn t).

    The paper's hash(e, i, t) is read as the mixed-radix index g = (e*N + i)*T + t,
    which cannot collide.  Ids outside their declared range are an error."""
    e, i, t = _i64(env_id), _i64(role_id), _i64(turn_id)
    if ((e < 0) | (e >= n_env) | (i < 0) | (i >= n_role) | (t < 0) | (t >= n_turn)).any():
        raise ValueError("group id out of range")
    return (e * n_role + i) * n_turn + t


def bucket_by_key(key, n_slots):
    """Collect the items that share a key (Sec. 4.1: data stored together under g).

    Returns (offsets[n_slots+1], perm[n_items]): slot s owns perm[offsets[s]:offsets[s+1]],
    listed in ascending item index (a stable counting sort).  Empty slots are allowed
    (an environment that terminated early leaves its later turns empty)."""
    key = _i64(key)
    if key.size and (key.min() < 0 or key.max() >= n_slots):
        raise ValueError("key out of range")
    counts = np.zeros(n_slots, dtype=np.int64)
    for k in key:                                   # histogram
        counts[k] += 1
    offsets = np.zeros(n_slots + 1, dtype=np.int64)
    for s in range(n_slots):                        # exclusive scan
        offsets[s + 1] = offsets[s] + counts[s]
    cursor = offsets[:-1].copy()
    perm = np.zeros(key.size, dtype=np.int64)
    for c in range(key.size):                       # stable placement, ascending item index
        perm[cursor[key[c]]] = c
        cursor[key[c]] += 1
    return offsets, perm


def group_advantages(rewards, key, n_slots, std_eps=1e-6, ddof=0):
    """Eq. 1: A(a^(c)) = (R(a^(c)) - mean_c R) / F_norm({R}) inside every group.

    F_norm = std + std_eps with std the (ddof) standard deviation of the group's K
    rewards, two-pass formula.  K = 1 gives A = 0.
    Returns (adv[n_cand], mean[n_slots], std[n_slots]); empty slots report mean = std = 0."""
    r = _f64(rewards)
    offsets, perm = bucket_by_key(key, n_slots)
    adv = np.zeros(r.size, dtype=np.float64)
    mean = np.zeros(n_slots, dtype=np.float64)
    std = np.zeros(n_slots, dtype=np.float64)
    for s in range(n_slots):
        members = perm[offsets[s]:offsets[s + 1]]
        K = members.size
        if K == 0:
            continue
        R = r[members]
        mu = R.sum() / K
        if K - ddof > 0:
            sd = np.sqrt(((R - mu) ** 2).sum() / (K - ddof))
        else:
            sd = 0.0
        mean[s], std[s] = mu, sd
        if K > 1:
            adv[members] = (R - mu) / (sd + std_eps)
    return adv, mean, std


def mix_rewards(r_team, r_loc, alpha=1.0):
    """Eq. 3: r_{t,i} = alpha * r_team_t + r_loc_{t,i}, per candidate.  The mixed reward is a
    float32 quantity (it is what Eq. 1 consumes), so the float64 sum is rounded to float32."""
    return (alpha * _f64(r_team) + _f64(r_loc)).astype(np.float32)


def group_argmax(rewards, key, n_slots):
    """Greedy selection of tree-structured sampling (Algorithm 1): for every group the candidate
    with the highest reward continues the rollout; ties go to the lowest candidate index; an empty
    slot reports -1."""
    r, key = _f64(rewards), _i64(key)
    best = np.full(n_slots, -1, dtype=np.int64)
    for c in range(r.size):                       # ascending index, strict '>' keeps the first maximum
        s = key[c]
        if best[s] < 0 or r[c] > r[best[s]]:
            best[s] = c
    return best


# --------------------------------------------------------------------------- routing
def route_tokens(role_of_token, head_of_role, n_heads):
    """Per-model batch B_m = union of D_i over the agents i with sigma(i) = m.

    role_of_token[j] is the agent i that produced response token j, head_of_role is
    sigma.  Returns (head_of_token, offsets[n_heads+1], perm[T]) with the tokens of
    head m listed in ascending token index."""
    role = _i64(role_of_token)
    sigma = _i64(head_of_role)
    if role.size and (role.min() < 0 or role.max() >= sigma.size):
        raise ValueError("role out of range")
    if sigma.size and (sigma.min() < 0 or sigma.max() >= n_heads):
        raise ValueError("head out of range")
    head = sigma[role] if role.size else np.zeros(0, dtype=np.int64)
    offsets, perm = bucket_by_key(head, n_heads)
    return head, offsets, perm


# --------------------------------------------------------------------------- LM head
def token_logprobs(H, W, target):
    """log pi_theta(y_j | .) for every response token j under one LM head.

    z_j = H_j W^T (all V logits), lse_j = log sum_v exp(z_jv),
    logp_j = z_{j, y_j} - lse_j.  Sampling temperature 1, no other term.
    Returns (lse[T], logp[T], z_target[T])."""
    H, W, y = _f64(H), _f64(W), _i64(target)
    if y.size and (y.min() < 0 or y.max() >= W.shape[0]):
        raise ValueError("target out of range")
    z = H @ W.T                                              # [T, V]
    zmax = z.max(axis=1)
    lse = zmax + np.log(np.exp(z - zmax[:, None]).sum(axis=1))
    zt = z[np.arange(y.size), y]
    return lse, zt - lse, zt


# --------------------------------------------------------------------------- Eq. 2
def clipped_objective(logp, old_logp, adv_of_token, eps_low=0.2, eps_high=0.2):
    """Per-token term of Eq. 2 (without the sign and the mean).

    r = pi_theta / pi_theta_old = exp(logp - old_logp);
    term = min(r*A, clip(r, 1-eps_low, 1+eps_high)*A).
    Also returns r and `active`, the indicator that d term / d r = A (the unclipped
    branch attains the min; ties pass the gradient; A = 0 is inactive)."""
    lp, lo, A = _f64(logp), _f64(old_logp), _f64(adv_of_token)
    r = np.exp(lp - lo)
    rc = np.minimum(np.maximum(r, 1.0 - eps_low), 1.0 + eps_high)
    unclipped, clipped = r * A, rc * A
    term = np.minimum(unclipped, clipped)
    active = (unclipped <= clipped) & (A != 0.0)
    return term, r, active


def policy_loss(logp, old_logp, adv, resp_of_token, head_of_token, n_heads,
                eps_low=0.2, eps_high=0.2):
    """Eq. 2 for every policy m: L_m = -(1/T_m) sum_{j in B_m} term_j.

    Token-level credit: token j carries the advantage of the response it belongs to,
    A = adv[resp_of_token[j]].  A policy with no token has loss 0.
    Returns (loss[n_heads], T_m[n_heads], clip_counts[n_heads, 2]) where clip_counts
    counts the tokens whose ratio lies below 1-eps_low / above 1+eps_high."""
    A = _f64(adv)[_i64(resp_of_token)]
    head = _i64(head_of_token)
    term, r, _ = clipped_objective(logp, old_logp, A, eps_low, eps_high)
    loss = np.zeros(n_heads, dtype=np.float64)
    count = np.zeros(n_heads, dtype=np.int64)
    clip_counts = np.zeros((n_heads, 2), dtype=np.int64)
    for m in range(n_heads):
        sel = head == m
        count[m] = sel.sum()
        if count[m]:
            loss[m] = -term[sel].sum() / count[m]
            clip_counts[m, 0] = (r[sel] < 1.0 - eps_low).sum()
            clip_counts[m, 1] = (r[sel] > 1.0 + eps_high).sum()
    return loss, count, clip_counts


def dloss_dlogp(logp, old_logp, adv, resp_of_token, head_of_token, n_heads, grad_loss=None,
                eps_low=0.2, eps_high=0.2):
    """c_j = d(sum_m grad_loss_m * L_m) / d logp_j = -grad_loss_m * A * r * active / T_m."""
    A = _f64(adv)[_i64(resp_of_token)]
    head = _i64(head_of_token)
    _, r, active = clipped_objective(logp, old_logp, A, eps_low, eps_high)
    count = np.bincount(head, minlength=n_heads).astype(np.float64)
    g = np.ones(n_heads) if grad_loss is None else _f64(grad_loss)
    denom = np.where(count > 0, count, 1.0)
    return -(g[head] / denom[head]) * A * r * active


def _sequence_terms(logp, old_logp, adv, resp_of_token, head_of_token, eps_low, eps_high):
    """Per response c that owns at least one token: r_c = pi(o_c|q)/pi_old(o_c|q) =
    exp(sum_j logp_j - sum_j old_logp_j) over its tokens, the Eq. 2 term, and its policy."""
    lp, lo = _f64(logp), _f64(old_logp)
    A_all = _f64(adv)
    resp, head = _i64(resp_of_token), _i64(head_of_token)
    ids = np.unique(resp)                                   # responses present in the batch
    delta = np.array([(lp[resp == c] - lo[resp == c]).sum() for c in ids])
    head_c = np.array([head[np.nonzero(resp == c)[0][0]] for c in ids], dtype=np.int64)
    term, r, active = clipped_objective(delta, np.zeros_like(delta), A_all[ids], eps_low, eps_high)
    return ids, head_c, term, r, active


def _response_weights(ids, head_c, n_heads, group_of_resp):
    """Weight of every present response in its policy's expectation, and the item count per policy.

    group_of_resp None: every response of policy m weighs 1/R_m (R_m = its responses with tokens).
    Otherwise Eq. 2's E_g[(1/K) sum_c .]: response c of group g weighs 1/(K_g * G_m), K_g = the
    responses of g that have tokens, G_m = the groups of policy m that have such a response."""
    w = np.zeros(ids.size)
    count = np.zeros(n_heads, dtype=np.int64)
    if group_of_resp is None:
        for m in range(n_heads):
            sel = head_c == m
            count[m] = sel.sum()
            if count[m]:
                w[sel] = 1.0 / count[m]
        return w, count
    grp = _i64(group_of_resp)[ids]
    for m in range(n_heads):
        groups = np.unique(grp[head_c == m])
        count[m] = groups.size
        for g in groups:
            members = (grp == g) & (head_c == m)
            w[members] = 1.0 / (members.sum() * groups.size)
    return w, count


def policy_loss_sequence(logp, old_logp, adv, resp_of_token, head_of_token, n_heads,
                         eps_low=0.2, eps_high=0.2, group_of_resp=None):
    """Eq. 2 read literally, with the sequence-level ratio r_c of every response c.

    group_of_resp None: L_m = -(1/R_m) sum_{responses c of policy m} min(r_c A_c, clip(r_c) A_c),
    R_m = the responses of policy m that have tokens.
    group_of_resp given (the group g of every response): the expectation exactly as printed,
    L_m = -(1/G_m) sum_g (1/K_g) sum_{c in g} min(...): every group counts once however many
    candidates it has (K varies when rollouts end early).
    Returns (loss[n_heads], count[n_heads] = R_m or G_m, clip_counts[n_heads, 2] per response)."""
    ids, head_c, term, r, _ = _sequence_terms(logp, old_logp, adv, resp_of_token, head_of_token,
                                              eps_low, eps_high)
    w, count = _response_weights(ids, head_c, n_heads, group_of_resp)
    loss = np.zeros(n_heads)
    cc = np.zeros((n_heads, 2), dtype=np.int64)
    for m in range(n_heads):
        sel = head_c == m
        if sel.any():
            loss[m] = -(w[sel] * term[sel]).sum()
            cc[m, 0] = (r[sel] < 1.0 - eps_low).sum()
            cc[m, 1] = (r[sel] > 1.0 + eps_high).sum()
    return loss, count, cc


def dloss_dlogp_sequence(logp, old_logp, adv, resp_of_token, head_of_token, n_heads, grad_loss=None,
                         eps_low=0.2, eps_high=0.2, group_of_resp=None):
    """c_j = d(sum_m grad_loss_m L_m)/d logp_j for the sequence-level loss: every token of response c
    gets -grad_loss_m * w_c * A_c * r_c * active_c (d r_c / d logp_j = r_c), w_c the response's
    weight in the expectation (1/R_m, or 1/(K_g G_m) with group_of_resp)."""
    ids, head_c, _, r, active = _sequence_terms(logp, old_logp, adv, resp_of_token, head_of_token,
                                                eps_low, eps_high)
    resp = _i64(resp_of_token)
    A_all = _f64(adv)
    g = np.ones(n_heads) if grad_loss is None else _f64(grad_loss)
    w, _ = _response_weights(ids, head_c, n_heads, group_of_resp)
    per_resp = {int(c): -g[h] * wc * A_all[c] * rc * ac for c, h, wc, rc, ac in zip(ids, head_c, w, r, active)}
    return np.array([per_resp[int(c)] for c in resp])


def policy_loss_grads(H, W_list, target, old_logp, adv, resp_of_token, head_of_token,
                      grad_loss=None, eps_low=0.2, eps_high=0.2, reduction="token", group_of_resp=None):
    """Gradient of sum_m grad_loss_m * L_m (Eq. 2) w.r.t. H and every head W_m.

    With c_j = dL/dlogp_j and p_jv = softmax(z_j)_v:
      dL/dz_jv = c_j * ([v = y_j] - p_jv)
      dH_j     = sum_v dL/dz_jv * W_m[v, :]      (m = head of token j)
      dW_m[v]  = sum_{j in B_m} dL/dz_jv * H_j
    Returns (dH[T, d], [dW_m[V, d]])."""
    Hd = _f64(H)
    y = _i64(target)
    head = _i64(head_of_token)
    M = len(W_list)
    logp = np.zeros(Hd.shape[0])
    P = [None] * M
    for m in range(M):
        sel = np.nonzero(head == m)[0]
        Wm = _f64(W_list[m])
        z = Hd[sel] @ Wm.T
        lse = np.log(np.exp(z - z.max(axis=1, keepdims=True)).sum(axis=1)) + z.max(axis=1)
        P[m] = np.exp(z - lse[:, None])
        logp[sel] = z[np.arange(sel.size), y[sel]] - lse
    if reduction == "token":
        c = dloss_dlogp(logp, old_logp, adv, resp_of_token, head, M, grad_loss, eps_low, eps_high)
    else:                                       # "sequence"; with group_of_resp the per-group mean
        c = dloss_dlogp_sequence(logp, old_logp, adv, resp_of_token, head, M, grad_loss, eps_low, eps_high,
                                 group_of_resp)
    dH = np.zeros_like(Hd)
    dW = []
    for m in range(M):
        sel = np.nonzero(head == m)[0]
        Wm = _f64(W_list[m])
        dz = -P[m] * c[sel][:, None]
        dz[np.arange(sel.size), y[sel]] += c[sel]
        dH[sel] = dz @ Wm
        dW.append(dz.T @ Hd[sel])
    return dH, dW


def policy_loss_grad_rows(H, W, target, lse, coef, token_rows=None, vocab_rows=None):
    """Selected rows of dH and dW for one head, from already-known lse and c_j = dL/dlogp_j.

    Same formulas as policy_loss_grads; used where the full [T,V] softmax does not fit:
    a dH row needs only that token's softmax, a dW row needs p_jv of one v for all j.
    `coef` is c_j of policy_loss_grads (sign included).  H, W, target, lse, coef all refer
    to the tokens of this head only."""
    Hd, Wd = _f64(H), _f64(W)
    y, lse, c = _i64(target), _f64(lse), _f64(coef)
    out_h = out_w = None
    if token_rows is not None:
        rows = _i64(token_rows)
        z = Hd[rows] @ Wd.T
        p = np.exp(z - lse[rows][:, None])
        dz = -p * c[rows][:, None]
        dz[np.arange(rows.size), y[rows]] += c[rows]
        out_h = dz @ Wd
    if vocab_rows is not None:
        vs = _i64(vocab_rows)
        z = Hd @ Wd[vs].T                                   # [T, n_v]
        p = np.exp(z - lse[:, None])
        dz = -p * c[:, None]
        dz += c[:, None] * (y[:, None] == vs[None, :])
        out_w = dz.T @ Hd
    return out_h, out_w


# --------------------------------------------------------------------------- parameter update
def grad_sumsq(grads):
    """Sum of squares of one policy's gradient tensors (the square of its global L2 norm)."""
    return float(sum((_f64(g) ** 2).sum() for g in grads))


def clip_scale(sumsq, max_norm):
    """Gradient clipping at max_norm: factor min(1, max_norm / (||g|| + 1e-6)); max_norm <= 0 = off."""
    if max_norm is None or max_norm <= 0:
        return 1.0
    return min(1.0, max_norm / (np.sqrt(sumsq) + 1e-6))


def adamw_step(theta, m, v, grad, step, lr=1e-6, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01,
               scale=1.0):
    """One AdamW step on one tensor (all float64): returns (theta, m, v) after step number `step` >= 1.

      g = scale * grad
      m = beta1*m + (1-beta1)*g            v = beta2*v + (1-beta2)*g^2
      theta = theta*(1 - lr*weight_decay) - lr * (m/(1-beta1^step)) / (sqrt(v/(1-beta2^step)) + eps)
    """
    theta, m, v, g = _f64(theta), _f64(m), _f64(v), _f64(grad) * scale
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    m_hat = m / (1.0 - beta1 ** step)
    v_hat = v / (1.0 - beta2 ** step)
    theta = theta * (1.0 - lr * weight_decay) - lr * m_hat / (np.sqrt(v_hat) + eps)
    return theta, m, v
