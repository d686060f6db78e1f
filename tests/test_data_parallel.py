"""Two-rank (gloo, CPU) check of the data-parallel plumbing: sharding by environment keeps groups
whole, and local results weighted by T_m(local)/T_m(global) and summed over ranks reproduce the
single-process oracle result."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    from oracle import atgrpo_oracle as O
    from paper_2510_11062_b200 import data_parallel as DP
    from paper_2510_11062_b200 import workloads as WL
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = WL.RolloutSpec("dp", 5, 3, 2, 4, (3, 3, 3), (9, 9, 9), 16, 50, 3, 321, 1)
    full = WL.make_rollout(spec)
    sh = DP.shard_batch_by_env(full, rank, world)
    G = spec.n_env * spec.n_role * spec.n_turn
    key = O.group_key(sh["env_id"], sh["role_id"], sh["turn_id"], spec.n_env, spec.n_role, spec.n_turn)
    adv, _, _ = O.group_advantages(sh["rewards"], key, G)
    head, _, _ = O.route_tokens(sh["role_of_token"], sh["head_of_role"], spec.n_heads)
    counts = torch.bincount(torch.from_numpy(head), minlength=spec.n_heads)
    scale, total = DP.token_mean_scale(counts)
    logp = np.zeros(sh["T"])
    for m in range(spec.n_heads):
        sel = head == m
        _, logp[sel], _ = O.token_logprobs(sh["H"][sel], sh["W"][m], sh["target"][sel])
    old = logp + 0.3 * np.cos(sh["token_index"].numpy())
    loss, _, _ = O.policy_loss(logp, old, adv, sh["resp_of_token"], head, spec.n_heads)
    dH, dW = O.policy_loss_grads(sh["H"], sh["W"], sh["target"], old, adv, sh["resp_of_token"], head,
                                 grad_loss=scale.numpy())
    wl = torch.from_numpy(loss) * scale.double()
    dist.all_reduce(wl)
    dWt = [torch.from_numpy(w) for w in dW]
    by_rows = [w.clone() for w in dWt]
    DP.allreduce_gradients(dWt)
    # the same sum taken row range by row range (what the overlapped backward does chunk by chunk)
    ranges = DP.chunk_row_ranges(spec.V, 4, 16)
    assert ranges == [(0, 16), (16, 32), (32, 48), (48, 50)]
    for lo, hi in ranges:
        DP.allreduce_gradient_rows(by_rows, lo, hi)
    assert all(torch.equal(a, b) for a, b in zip(by_rows, dWt))
    q.put((rank, adv, sh["token_index"].numpy(), dH, wl.numpy(), [w.numpy() for w in dWt], total.numpy(),
           np.nonzero(((full["env_id"] % world) == rank).numpy())[0]))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_rank_sharding_matches_single_process():
    sys.path.insert(0, ROOT)
    from oracle import atgrpo_oracle as O
    from paper_2510_11062_b200 import workloads as WL
    world, port = 2, 29531 + os.getpid() % 500
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted([q.get(timeout=100) for _ in range(world)], key=lambda x: x[0])
    for p in procs:
        p.join(30)
        assert p.exitcode == 0
    spec = WL.RolloutSpec("dp", 5, 3, 2, 4, (3, 3, 3), (9, 9, 9), 16, 50, 3, 321, 1)
    full = WL.make_rollout(spec)
    G = spec.n_env * spec.n_role * spec.n_turn
    key = O.group_key(full["env_id"], full["role_id"], full["turn_id"], spec.n_env, spec.n_role, spec.n_turn)
    adv, _, _ = O.group_advantages(full["rewards"], key, G)
    head, _, _ = O.route_tokens(full["role_of_token"], full["head_of_role"], spec.n_heads)
    logp = np.zeros(full["T"])
    for m in range(spec.n_heads):
        sel = head == m
        _, logp[sel], _ = O.token_logprobs(full["H"][sel], full["W"][m], full["target"][sel])
    old = logp + 0.3 * np.cos(np.arange(full["T"]))
    loss, count, _ = O.policy_loss(logp, old, adv, full["resp_of_token"], head, spec.n_heads)
    dH, dW = O.policy_loss_grads(full["H"], full["W"], full["target"], old, adv, full["resp_of_token"], head)
    seen = np.zeros(full["T"], bool)
    for rank, adv_r, tok_idx, dH_r, wl, dW_r, total, cand_idx in res:
        np.testing.assert_allclose(adv_r, adv[cand_idx], atol=1e-15)          # groups stayed whole
        np.testing.assert_allclose(dH_r, dH[tok_idx], rtol=1e-6, atol=1e-14)   # scale is fp32
        np.testing.assert_allclose(wl, loss, rtol=1e-6, atol=1e-14)                      # global token mean
        for m in range(spec.n_heads):
            np.testing.assert_allclose(dW_r[m], dW[m], rtol=1e-6, atol=1e-8)
        assert (total == count).all()
        assert not seen[tok_idx].any()
        seen[tok_idx] = True
    assert seen.all()
