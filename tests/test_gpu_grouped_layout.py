"""Grouped advantage on candidates whose groups are adjacent (params.candidates_grouped = 1, the
order Algorithm 1 appends them in) vs. the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu


def _ids(slot, n_role, n_turn):
    env_id = (slot // (n_role * n_turn)).to(torch.int32)
    role_id = ((slot // n_turn) % n_role).to(torch.int32)
    turn_id = (slot % n_turn).to(torch.int32)
    return env_id, role_id, turn_id


def _check(rewards, env_id, role_id, turn_id, n_env, n_role, n_turn, ddof=0):
    prm = A.Params(ddof=ddof, candidates_grouped=1)
    ref = U.oracle_group_advantages(rewards, env_id, role_id, turn_id, n_env, n_role, n_turn, ddof=ddof)
    gpu = U.gpu_group_advantages(rewards, env_id, role_id, turn_id, n_env, n_role, n_turn, prm, bucketing=False)
    U.check_group_advantages(gpu, ref)
    return gpu, ref


@pytest.mark.parametrize("name", ["tiny", "multi3", "qwen3_8b"])
def test_rollout_batches_are_grouped(name):
    # rollout order is (environment, turn, role, candidate): groups adjacent, group ids not monotone
    b = WL.make_rollout(WL.SPECS[name], with_weights=False)
    s = b["spec"]
    _check(b["rewards"], b["env_id"], b["role_id"], b["turn_id"], s.n_env, s.n_role, s.n_turn)


@pytest.mark.parametrize("ddof", [0, 1])
def test_stress_shape_in_rollout_order(ddof):
    # K ~ U{1..16} with K = 1 and all-equal groups; several tiles of 4096 candidates and a ragged tail
    s = WL.make_stress(n_env=519, n_role=4, n_turn=4, n_tokens=10, seed=5, shuffle=False)
    assert s["R"] > 4 * 4096 and s["R"] % 4096 != 0
    _check(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 519, 4, 4, ddof=ddof)


def test_groups_in_random_order_with_empty_slots():
    g = torch.Generator().manual_seed(11)
    G = 700
    sizes = torch.randint(0, 9, (G,), generator=g)
    order = torch.randperm(G, generator=g)
    slot = torch.repeat_interleave(order, sizes[order])
    rewards = WL.draw_rewards(g, slot.numel())
    e, r, t = _ids(slot, 5, 2)
    _check(rewards, e, r, t, 70, 5, 2)


@pytest.mark.parametrize("shift", [0, 1, 1791, 2047, 3839, 4095])
def test_runs_that_cross_tiles_and_outgrow_the_window(shift):
    # runs of 9000 (spans whole tiles), 4352 and 257 (just beyond the look-ahead), 256, 255 members,
    # placed so that they start at different offsets inside a 4096-candidate tile (4096 + 256 staged)
    g = torch.Generator().manual_seed(3)
    sizes = [shift, 9000, 3, 4352, 1, 257, 256, 255, 4090, 2304, 700, 65, 33] + [3] * 50 + [1] * 7 + [0] * 5
    slot = torch.repeat_interleave(torch.arange(len(sizes)), torch.tensor(sizes))
    rewards = WL.draw_rewards(g, slot.numel())
    e, r, t = _ids(slot, 3, 2)
    _check(rewards, e, r, t, 14, 3, 2)
    _check(rewards, e, r, t, 14, 3, 2, ddof=1)


def test_unaligned_pointers_take_the_scalar_staging_path():
    s = WL.make_stress(n_env=300, n_role=2, n_turn=2, n_tokens=10, seed=8, shuffle=False)
    R = s["R"]
    assert R > 2 * 4096
    pad = lambda t: torch.cat([torch.zeros(1, dtype=t.dtype), t]).to(U.DEV)[1:]   # 4-byte aligned only
    rewards, e, r, t = pad(s["rewards"]), pad(s["env_id"]), pad(s["role_id"]), pad(s["turn_id"])
    adv = torch.empty(R + 1, dtype=torch.float32, device=U.DEV)[1:]
    gid = torch.empty(R + 1, dtype=torch.int32, device=U.DEV)[1:]
    status = A.new_status(U.DEV)
    ws = A.workspace(A.atgrpo_group_advantages_workspace_bytes(R, 1200), U.DEV)
    A.atgrpo_group_advantages(rewards, e, r, t, 300, 2, 2, A.Params(candidates_grouped=1), adv, group_of_cand=gid,
                              device_status=status, workspace=ws)
    torch.cuda.synchronize()
    ref = U.oracle_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 300, 2, 2)
    U.check_group_advantages(dict(adv=adv.cpu(), group_of_cand=gid.cpu(), status=int(status.item())), ref)


def test_single_candidate_and_constant_long_run():
    one = torch.zeros(1, dtype=torch.int32)
    gpu, _ = _check(torch.tensor([0.7]), one, one, one, 1, 1, 1)
    assert gpu["adv"].tolist() == [0.0]
    n = 9000                                     # one constant run longer than the staged window
    z = torch.zeros(n, dtype=torch.int32)
    gpu, _ = _check(torch.full((n,), 0.3), z, z, z, 1, 1, 1)
    assert (gpu["adv"] == 0).all()


def test_nearly_equal_and_wide_range_rewards_in_adjacent_groups():
    # groups whose rewards differ in the last bit, negative rewards, magnitudes from 1e-20 to 1e20 next
    # to one another: every run is shifted by its own first reward, and squares beyond fp32 take fp64
    one = torch.tensor(1.0)
    up = torch.nextafter(one, torch.tensor(2.0))
    rewards = torch.tensor([1.0, up, 1.0, up, -3.0, -3.0, -3.0, -2.9999998, 1e-20, 3e-20, 2e-20, 5e20, -5e20, 0.0,
                            7.5, 2e19, -2e19, 1e19, 4.0, 4.0, 4.0], dtype=torch.float32)
    slot = torch.tensor([0, 0, 0, 0, 1, 1, 1, 1, 2, 2, 2, 3, 3, 3, 4, 5, 5, 5, 6, 6, 6])
    env = slot.to(torch.int32)
    zero = torch.zeros_like(env)
    for ddof in (0, 1):
        gpu, ref = _check(rewards, env, zero, zero, 7, 1, 1, ddof=ddof)
    assert (gpu["adv"][-3:] == 0).all() and gpu["adv"][14] == 0


@pytest.mark.parametrize("scale", [1e-18, 1e18])
def test_rewards_of_extreme_scale_with_an_epsilon_to_match(scale):
    # rewards around 1e-18 (squared deviations fall into the fp32 denormal range) and around 1e18 (they
    # overflow fp32), with std_eps scaled alike so that it does not mask the standard deviation
    s = WL.make_stress(n_env=200, n_role=2, n_turn=2, n_tokens=10, seed=12, shuffle=False)
    rewards = (s["rewards"] * scale).contiguous()
    eps = 1e-6 * scale
    args = (rewards, s["env_id"], s["role_id"], s["turn_id"], 200, 2, 2)
    ref = U.oracle_group_advantages(*args, eps=eps)
    gpu = U.gpu_group_advantages(*args, A.Params(std_eps=eps, candidates_grouped=1), bucketing=False)
    assert gpu["status"] == 0
    a, r = gpu["adv"].numpy().astype(np.float64), ref["adv"]
    assert (np.abs(a - r) <= 1e-5 * np.maximum(1.0, np.abs(r))).all()
    assert (a[r == 0.0] == 0.0).all()
    np.testing.assert_allclose(gpu["group_std"].numpy(), ref["group_std"], rtol=2e-6)


def test_bad_ids_inside_and_between_runs():
    rewards = torch.tensor([0.1, 0.9, 0.5, 0.3, 0.2, 0.8, 0.4], dtype=torch.float32)
    env = torch.tensor([0, 0, 5, 0, 1, -1, 1], dtype=torch.int32)      # a bad id splits group 0 and group 1
    zero = torch.zeros(7, dtype=torch.int32)
    prm = A.Params(candidates_grouped=1)
    gpu = U.gpu_group_advantages(rewards, env, zero, zero, 2, 1, 1, prm, bucketing=False)
    # the bad ids are reported first or the split groups are: either way the call is flagged, the bad
    # candidates get 0 and every stretch gets its own statistics
    assert gpu["status"] in (A.ERR_BAD_INDEX, A.ERR_LAYOUT)
    assert gpu["adv"][2] == 0 and gpu["adv"][5] == 0
    ref = U.oracle_group_advantages(rewards[:2], env[:2], zero[:2], zero[:2], 2, 1, 1)
    np.testing.assert_allclose(gpu["adv"].numpy()[:2], ref["adv"], rtol=1e-5)
    assert gpu["adv"][3] == 0 and gpu["adv"][4] == 0 and gpu["adv"][6] == 0       # stretches of one member


def test_broken_promise_is_flagged():
    s = WL.make_stress(n_env=64, n_role=2, n_turn=2, n_tokens=10, seed=9)        # shuffled candidates
    prm = A.Params(candidates_grouped=1)
    gpu = U.gpu_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 64, 2, 2, prm,
                                 bucketing=False)
    assert gpu["status"] == A.ERR_LAYOUT
    assert torch.isfinite(gpu["adv"]).all()
    # with bucketing outputs requested the flag is ignored and the general pipeline runs
    ref = U.oracle_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 64, 2, 2)
    gpu = U.gpu_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 64, 2, 2, prm)
    U.check_group_advantages(gpu, ref)


def test_full_size_stress_in_rollout_order():
    # 262144 slots, 2.23 M candidates in the launch configuration the benchmark times: every
    # candidate, group id, group mean and std against the fp64 oracle
    s = WL.make_stress(shuffle=False)
    args = (s["rewards"], s["env_id"], s["role_id"], s["turn_id"], s["n_env"], s["n_role"], s["n_turn"])
    ref = U.oracle_group_advantages(*args)
    fast = U.gpu_group_advantages(*args, A.Params(candidates_grouped=1), bucketing=False)
    U.check_group_advantages(fast, ref)
    assert (ref["adv"] == 0).sum() > 0.01 * s["G"]
    again = U.gpu_group_advantages(*args, A.Params(candidates_grouped=1), bucketing=False)
    assert torch.equal(fast["adv"], again["adv"])                  # bit-reproducible


def _packed(s, prm, bucketing=False, device_slice=None):
    dev = U.DEV
    R, G = s["R"], s["G"]
    out = dict(adv=torch.full((R,), 7.0, device=dev), group_mean=torch.full((G,), 7.0, device=dev),
               group_std=torch.full((G,), 7.0, device=dev))
    if bucketing:
        out.update(group_offsets=torch.full((G + 1,), -5, dtype=torch.int32, device=dev),
                   group_perm=torch.full((R,), -5, dtype=torch.int32, device=dev))
    st = A.new_status(dev)
    ws = A.workspace(A.atgrpo_group_advantages_workspace_bytes(R, G), dev)
    A.atgrpo_group_advantages_packed(s["rewards"].to(dev), s["group_id"].to(dev), G, prm, device_status=st,
                                     workspace=ws, **out)
    torch.cuda.synchronize()
    res = {k: v.cpu() for k, v in out.items()}
    res["status"] = int(st.item())
    return res


@pytest.mark.parametrize("shuffle,grouped,bucketing", [(False, 1, False), (True, 0, False), (True, 0, True)])
def test_packed_group_ids_take_every_pipeline(shuffle, grouped, bucketing):
    # one dense group id per candidate instead of the three id arrays: the streaming pass on
    # adjacent groups, the sort-free pipeline and the counting sort, each against the oracle
    s = WL.make_stress(n_env=519, n_role=4, n_turn=4, n_tokens=10, seed=6, shuffle=shuffle)
    ref = U.oracle_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 519, 4, 4)
    assert np.array_equal(ref["group_of_cand"], s["group_id"].numpy())          # the generator's slot IS the key
    got = _packed(s, A.Params(candidates_grouped=grouped), bucketing=bucketing)
    U.check_group_advantages(got, ref)


def test_packed_group_id_out_of_range_is_flagged():
    s = WL.make_stress(n_env=40, n_role=2, n_turn=2, n_tokens=10, seed=7, shuffle=False)
    s["group_id"] = s["group_id"].clone()
    s["group_id"][5] = s["G"] + 3
    got = _packed(s, A.Params(candidates_grouped=1))
    assert got["status"] in (A.ERR_BAD_INDEX, A.ERR_LAYOUT) and got["adv"][5] == 0
