"""Eq. 3 reward mix + Eq. 1 advantages + greedy per-group argmax on the GPU vs. the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import atgrpo_oracle as O
from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu


def _run(team, loc, alpha, env, role, turn, dims):
    dev = U.DEV
    R, G = team.numel(), dims[0] * dims[1] * dims[2]
    f32, i32 = torch.float32, torch.int32
    out = dict(rewards_out=torch.full((R,), 7.0, dtype=f32, device=dev), adv=torch.full((R,), 7.0, dtype=f32, device=dev),
               group_best=torch.full((G,), -5, dtype=i32, device=dev),
               group_mean=torch.full((G,), 7.0, dtype=f32, device=dev),
               group_std=torch.full((G,), 7.0, dtype=f32, device=dev))
    st = A.new_status(dev)
    ws = A.workspace(A.atgrpo_group_select_workspace_bytes(R, G), dev)
    A.atgrpo_group_select(team.to(dev), loc.to(dev), alpha, env.to(dev), role.to(dev), turn.to(dev), *dims, A.Params(),
                          device_status=st, workspace=ws, **out)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return {k: v.cpu() for k, v in out.items()}


@pytest.mark.parametrize("alpha", [1.0, 0.37])
def test_mix_advantages_and_argmax(alpha):
    s = WL.make_stress(n_env=700, n_role=4, n_turn=4, n_tokens=10, seed=41)
    R, dims = s["R"], (700, 4, 4)
    g = torch.Generator().manual_seed(4)
    team = (torch.rand(R, generator=g) < 0.5).float()
    loc = torch.rand(R, generator=g)
    out = _run(team, loc, alpha, s["env_id"], s["role_id"], s["turn_id"], dims)
    mixed = O.mix_rewards(team, loc, alpha)
    got = out["rewards_out"].numpy()
    assert np.abs(got - mixed).max() <= 1.2e-7 * np.abs(mixed).max()        # at most one fp32 ulp (double rounding)
    key = O.group_key(s["env_id"], s["role_id"], s["turn_id"], *dims)
    G = dims[0] * dims[1] * dims[2]
    adv, mean, std = O.group_advantages(mixed, key, G)
    a = out["adv"].numpy().astype(np.float64)
    assert (np.abs(a - adv) <= 1e-5 * np.maximum(1.0, np.abs(adv))).all()
    np.testing.assert_allclose(out["group_mean"].numpy(), mean, rtol=1e-6, atol=1e-7)
    best = O.group_argmax(mixed, key, G)
    gb = out["group_best"].numpy().astype(np.int64)
    assert ((gb < 0) == (best < 0)).all()
    # the selection is unique where the top two rewards differ by more than an ulp; elsewhere it must be valid
    same = gb == best
    bad = np.nonzero(~same)[0]
    for s_ in bad:
        assert key[gb[s_]] == s_ and abs(mixed[gb[s_]] - mixed[best[s_]]) <= 1.2e-7 * max(1.0, abs(mixed[best[s_]]))
    assert same.mean() > 0.999


def test_argmax_ties_go_to_the_lowest_index_and_empty_slots():
    team = torch.tensor([0.5, 0.5, 0.5, 0.0, 1.0, 1.0], dtype=torch.float32)
    loc = torch.tensor([0.25, 0.25, 0.125, 0.75, 0.0, 0.0], dtype=torch.float32)
    env = torch.tensor([0, 0, 0, 0, 2, 2], dtype=torch.int32)
    z = torch.zeros(6, dtype=torch.int32)
    out = _run(team, loc, 1.0, env, z, z, (4, 1, 1))
    assert out["group_best"].tolist() == [0, -1, 4, -1]           # 0.75 three times in group 0: lowest index wins
    assert out["rewards_out"].tolist() == [0.75, 0.75, 0.625, 0.75, 1.0, 1.0]
