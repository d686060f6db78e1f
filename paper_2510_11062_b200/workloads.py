"""Seeded synthetic workloads for the AT-GRPO policy-update path.

This module only draws inputs; it holds none of the method's arithmetic (no
advantage, log-prob, ratio or loss formula).  The same CPU tensors are handed to
the CUDA library and to any checker.  Shapes follow the five workloads the
library is measured on: a tiny single-policy case, two Qwen3-shaped single-policy
LM heads (d=2048 and d=4096, V=151936), a three-role multi-policy case, and a
memory-bound grouping stress case.  They stand in for the paper's game / planning
/ code / math rollouts (Sec. 5): only the structure is kept -- E environments,
N roles, T turns, K sampled candidates per (environment, role, turn), response
lengths in tokens -- never any dataset item.

All draws come from one torch.Generator seeded per workload, in a fixed order, on
the CPU; bf16 rounding (round-to-nearest-even) happens once, here.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

__all__ = ["RolloutSpec", "SPECS", "make_rollout", "make_old_logp", "make_stress", "draw_rewards"]


@dataclass(frozen=True)
class RolloutSpec:
    name: str
    n_env: int
    n_role: int
    n_turn: int
    K: int
    len_lo: tuple          # per-role inclusive lower bound of the response length
    len_hi: tuple          # per-role inclusive upper bound
    d: int
    V: int
    n_heads: int           # 1 = shared policy (M=1), n_role = one head per role (M=N)
    seed: int
    n_const_groups: int = 2


SPECS = {
    # tiny single-policy
    "tiny": RolloutSpec("tiny", 4, 2, 2, 4, (16, 16), (64, 64), 128, 2048, 1, 1235),
    # single policy, Qwen3-1.7B-shaped head
    "qwen3_1p7b": RolloutSpec("qwen3_1p7b", 16, 2, 2, 4, (32, 32), (96, 96), 2048, 151936, 1, 1236),
    # the same head on a quarter of the batch: small enough for multi-pass profiler captures
    "qwen3_1p7b_small": RolloutSpec("qwen3_1p7b_small", 4, 2, 2, 4, (32, 32), (96, 96), 2048, 151936, 1, 1242),
    # three roles, one head per role, role 0 carries about half of the tokens
    "multi3": RolloutSpec("multi3", 24, 3, 2, 4, (96, 32, 32), (128, 80, 80), 2048, 151936, 3, 1237),
    # single policy, Qwen3-8B-shaped head
    "qwen3_8b": RolloutSpec("qwen3_8b", 32, 2, 4, 4, (16, 16), (48, 48), 4096, 151936, 1, 1238),
    # the same head on a quarter of the batch (~8K tokens): dense parity at d = 4096 within the oracle's reach
    "qwen3_8b_quarter": RolloutSpec("qwen3_8b_quarter", 8, 2, 4, 4, (16, 16), (48, 48), 4096, 151936, 1, 1244),
    # long responses (the paper allows up to 4096 generated tokens): few responses, ~80K tokens
    "long_resp": RolloutSpec("long_resp", 4, 2, 2, 4, (512, 512), (2048, 2048), 2048, 151936, 1, 1243),
    # mid-size shapes for dense element-by-element comparison (several tiles + ragged tails)
    "mid": RolloutSpec("mid", 6, 2, 2, 4, (8, 8), (40, 40), 256, 8192 + 72, 1, 1240),
    "mid_multi": RolloutSpec("mid_multi", 6, 3, 2, 4, (24, 8, 8), (40, 24, 24), 192, 4096 + 40, 3, 1241),
}


def draw_rewards(gen: torch.Generator, n: int) -> torch.Tensor:
    """reward = 0.5 * Bernoulli(0.5) team part + 0.5 * U[0,1] role part, per candidate, fp32."""
    team = (torch.rand(n, generator=gen, dtype=torch.float32) < 0.5).to(torch.float32)
    local = torch.rand(n, generator=gen, dtype=torch.float32)
    return 0.5 * team + 0.5 * local


def make_rollout(spec: RolloutSpec, scale_H: float = 1.0, with_weights: bool = True) -> dict:
    """One on-policy batch as Phase 1 of Algorithm 1 would leave it.

    Responses are laid out environment-major (env, turn, role, candidate), so the
    roles are interleaved and never globally contiguous.  Every response is one
    candidate of its (env, role, turn) group.  Returns CPU tensors:
      rewards f32[R], env_id/role_id/turn_id i32[R], resp_len i32[R],
      resp_of_token i32[T], role_of_token i32[T], head_of_role i32[n_role],
      H bf16[T,d], W list of bf16[V,d], target i32[T].
    """
    g = torch.Generator(device="cpu")
    g.manual_seed(spec.seed)
    E, N, Tn, K = spec.n_env, spec.n_role, spec.n_turn, spec.K
    env, role, turn = [], [], []
    for e in range(E):
        for t in range(Tn):
            for i in range(N):
                for _ in range(K):
                    env.append(e), role.append(i), turn.append(t)
    R = len(env)
    env_id = torch.tensor(env, dtype=torch.int32)
    role_id = torch.tensor(role, dtype=torch.int32)
    turn_id = torch.tensor(turn, dtype=torch.int32)
    lo = torch.tensor(spec.len_lo, dtype=torch.int64)[role_id.long()]
    hi = torch.tensor(spec.len_hi, dtype=torch.int64)[role_id.long()]
    u = torch.rand(R, generator=g, dtype=torch.float64)
    resp_len = (lo + torch.floor(u * (hi - lo + 1).double()).long()).clamp(max=hi).to(torch.int32)
    rewards = draw_rewards(g, R)
    # a few groups get identical rewards (all candidates tie)
    n_groups = E * N * Tn
    const_groups = torch.randperm(n_groups, generator=g)[: spec.n_const_groups]
    const_vals = torch.rand(spec.n_const_groups, generator=g, dtype=torch.float32)
    for cg, cv in zip(const_groups.tolist(), const_vals.tolist()):
        e, rest = divmod(cg, N * Tn)
        i, t = divmod(rest, Tn)
        rewards[(env_id == e) & (role_id == i) & (turn_id == t)] = cv
    resp_of_token = torch.repeat_interleave(torch.arange(R, dtype=torch.int32), resp_len.long())
    role_of_token = role_id[resp_of_token.long()].contiguous()
    T = int(resp_of_token.numel())
    head_of_role = (torch.arange(N, dtype=torch.int32) if spec.n_heads > 1
                    else torch.zeros(N, dtype=torch.int32))
    out = dict(spec=spec, rewards=rewards, env_id=env_id, role_id=role_id, turn_id=turn_id,
               resp_len=resp_len, resp_of_token=resp_of_token, role_of_token=role_of_token,
               head_of_role=head_of_role, T=T, R=R)
    out["target"] = torch.randint(0, spec.V, (T,), generator=g, dtype=torch.int64).to(torch.int32)
    if with_weights:
        H = torch.randn(T, spec.d, generator=g, dtype=torch.float32) * scale_H
        out["H"] = H.to(torch.bfloat16)
        W = []
        for _ in range(spec.n_heads):
            w = torch.randn(spec.V, spec.d, generator=g, dtype=torch.float32) * (spec.d ** -0.5)
            W.append(w.to(torch.bfloat16))
        out["W"] = W
    return out


def make_old_logp(logp: torch.Tensor, seed: int, sigma: float = 0.05) -> torch.Tensor:
    """old_logp = logp + N(0, sigma), fp32.  `logp` is whatever log-probabilities the caller
    supplies (a checker's, or the library's own for perf-only runs)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    noise = torch.randn(logp.numel(), generator=g, dtype=torch.float32) * sigma
    return (logp.detach().to("cpu", torch.float32) + noise).contiguous()


def make_stress(n_env: int = 16384, n_role: int = 4, n_turn: int = 4, k_max: int = 16,
                n_tokens: int = 4_194_304, seed: int = 1239, frac_const: float = 0.01,
                exact_R: int | None = None, shuffle: bool = True) -> dict:
    """Memory-bound grouping + loss-reduction stress input.

    G = n_env*n_role*n_turn group slots, group sizes K_g ~ U{1..k_max} (K=1 groups occur
    naturally), candidates globally shuffled, at least frac_const of the groups given
    identical rewards.  With shuffle=False the candidates stay in rollout order instead (the
    members of a group adjacent, as Algorithm 1 appends them).  With exact_R the groups are filled in slot order until exactly
    exact_R candidates exist (later slots stay empty).  Tokens: n_tokens response tokens,
    resp_of_token = sorted U{0..R-1} (responses of length 0 allowed), logp ~ U[-12,-0.1],
    old_logp = logp + N(0, 0.05)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    G = n_env * n_role * n_turn
    Kg = torch.randint(1, k_max + 1, (G,), generator=g, dtype=torch.int64)
    if exact_R is not None:
        csum = torch.cumsum(Kg, 0)
        over = csum > exact_R
        Kg = torch.where(over, (exact_R - (csum - Kg)).clamp(min=0), Kg)
    slot = torch.repeat_interleave(torch.arange(G, dtype=torch.int64), Kg)
    R = int(slot.numel())
    rewards = draw_rewards(g, R)
    n_const = max(1, int(frac_const * G))
    const_groups = torch.randperm(G, generator=g)[:n_const]
    const_vals = torch.rand(G, generator=g, dtype=torch.float32)
    is_const = torch.zeros(G, dtype=torch.bool)
    is_const[const_groups] = True
    rewards = torch.where(is_const[slot], const_vals[slot], rewards)
    order = torch.randperm(R, generator=g)
    if shuffle:
        slot, rewards = slot[order], rewards[order].contiguous()
    turn_id = (slot % n_turn).to(torch.int32)
    role_id = ((slot // n_turn) % n_role).to(torch.int32)
    env_id = (slot // (n_turn * n_role)).to(torch.int32)
    resp_of_token = torch.sort(torch.randint(0, R, (n_tokens,), generator=g, dtype=torch.int64)).values
    logp = (torch.rand(n_tokens, generator=g, dtype=torch.float32) * 11.9 - 12.0)
    old_logp = logp + torch.randn(n_tokens, generator=g, dtype=torch.float32) * 0.05
    return dict(rewards=rewards, env_id=env_id, role_id=role_id, turn_id=turn_id,
                group_id=slot.to(torch.int32),       # the slot each candidate was drawn for, as one dense id
                n_env=n_env, n_role=n_role, n_turn=n_turn, R=R, G=G,
                resp_of_token=resp_of_token.to(torch.int32), logp=logp, old_logp=old_logp,
                T=n_tokens)
