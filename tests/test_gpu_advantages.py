"""CUDA grouped advantage and Eq. 2 reduction vs. the fp64 oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

from oracle import atgrpo_oracle as O
from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu


def _run_case(rewards, env_id, role_id, turn_id, n_env, n_role, n_turn, ddof=0):
    prm = A.Params(ddof=ddof)
    ref = U.oracle_group_advantages(rewards, env_id, role_id, turn_id, n_env, n_role, n_turn, ddof=ddof)
    for bucketing in (False, True):          # sort-free pipeline, then counting-sort pipeline
        gpu = U.gpu_group_advantages(rewards, env_id, role_id, turn_id, n_env, n_role, n_turn, prm,
                                     bucketing=bucketing)
        U.check_group_advantages(gpu, ref)
    return gpu, ref


@pytest.mark.parametrize("name", ["tiny", "multi3", "qwen3_8b"])
def test_rollout_groups(name):
    b = WL.make_rollout(WL.SPECS[name], with_weights=False)
    s = b["spec"]
    gpu, ref = _run_case(b["rewards"], b["env_id"], b["role_id"], b["turn_id"], s.n_env, s.n_role, s.n_turn)
    assert (ref["adv"] == 0).sum() >= 4 * s.n_const_groups


@pytest.mark.parametrize("ddof", [0, 1])
def test_stress_shape_reduced(ddof):
    # same structure as the 262144-group stress input (shuffled, K ~ U{1..16}, K=1 and all-equal
    # groups), at a size the pure-Python oracle finishes in seconds; several blocks + ragged tail
    s = WL.make_stress(n_env=519, n_role=4, n_turn=4, n_tokens=1000, seed=5)
    _run_case(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 519, 4, 4, ddof=ddof)


def test_stress_exact_R_with_empty_slots():
    s = WL.make_stress(n_env=300, n_role=4, n_turn=4, n_tokens=10, seed=6, exact_R=20000)
    assert s["R"] == 20000
    _run_case(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 300, 4, 4)


def test_large_groups_take_the_block_path():
    g = torch.Generator().manual_seed(3)
    # group sizes: one of 6000 (ordered rescan), one of 700 (shared-memory sort), many small, unaligned R
    sizes = [6000, 700, 65, 33] + [3] * 50 + [1] * 7 + [0] * 5
    slot = torch.repeat_interleave(torch.arange(len(sizes)), torch.tensor(sizes))
    R = slot.numel()
    perm = torch.randperm(R, generator=g)
    slot = slot[perm]
    rewards = WL.draw_rewards(g, R)
    n_env, n_role, n_turn = 11, 3, 2
    assert n_env * n_role * n_turn >= len(sizes)
    env_id = (slot // (n_role * n_turn)).to(torch.int32)
    role_id = ((slot // n_turn) % n_role).to(torch.int32)
    turn_id = (slot % n_turn).to(torch.int32)
    _run_case(rewards, env_id, role_id, turn_id, n_env, n_role, n_turn)


def test_nearly_equal_and_wide_range_rewards():
    # groups whose rewards differ in the last bit, negative rewards, and magnitudes from 1e-20 to 1e20:
    # a sum-of-squares formula without a shift would lose these
    one = torch.tensor(1.0)
    up = torch.nextafter(one, torch.tensor(2.0))
    rewards = torch.tensor([1.0, up, 1.0, up, -3.0, -3.0, -3.0, -2.9999998, 1e-20, 3e-20, 2e-20, 5e20, -5e20, 0.0,
                            7.5], dtype=torch.float32)
    slot = torch.tensor([0, 0, 0, 0, 1, 1, 1, 1, 2, 2, 2, 3, 3, 3, 4])
    env = slot.to(torch.int32)
    zero = torch.zeros_like(env)
    _run_case(rewards, env, zero, zero, 5, 1, 1)
    _run_case(rewards, env, zero, zero, 5, 1, 1, ddof=1)


def test_unaligned_pointers_and_no_optional_outputs():
    s = WL.make_stress(n_env=40, n_role=2, n_turn=2, n_tokens=10, seed=8)
    R = s["R"]
    dev = U.DEV
    pad = lambda t: torch.cat([torch.zeros(1, dtype=t.dtype), t]).to(dev)[1:]   # 4-byte aligned only
    rewards, e, r, t = pad(s["rewards"]), pad(s["env_id"]), pad(s["role_id"]), pad(s["turn_id"])
    adv = torch.empty(R, dtype=torch.float32, device=dev)
    status = A.new_status(dev)
    ws = A.workspace(A.atgrpo_group_advantages_workspace_bytes(R, 160), dev)
    A.atgrpo_group_advantages(rewards, e, r, t, 40, 2, 2, A.Params(), adv, device_status=status, workspace=ws)
    torch.cuda.synchronize()
    ref = U.oracle_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 40, 2, 2)
    U.check_group_advantages(dict(adv=adv.cpu(), status=int(status.item())), ref)


def test_empty_input_and_bad_ids():
    dev = U.DEV
    z_f = torch.zeros(0, dtype=torch.float32, device=dev)
    z_i = torch.zeros(0, dtype=torch.int32, device=dev)
    off = torch.full((9,), -1, dtype=torch.int32, device=dev)
    ws = A.workspace(A.atgrpo_group_advantages_workspace_bytes(0, 8), dev)
    A.atgrpo_group_advantages(z_f, z_i, z_i, z_i, 2, 2, 2, A.Params(), z_f, group_offsets=off,
                              device_status=A.new_status(dev), workspace=ws)
    torch.cuda.synchronize()
    assert (off == 0).all()
    # an id out of range: flagged on the device, that candidate gets 0 and joins no group
    rewards = torch.tensor([0.1, 0.9, 0.5, 0.3], dtype=torch.float32)
    env = torch.tensor([0, 0, 5, 0], dtype=torch.int32)
    zero = torch.zeros(4, dtype=torch.int32)
    gpu = U.gpu_group_advantages(rewards, env, zero, zero, 2, 1, 1)
    assert gpu["status"] == A.ERR_BAD_INDEX
    ref = U.oracle_group_advantages(rewards[[0, 1, 3]], env[[0, 1, 3]], zero[:3], zero[:3], 2, 1, 1)
    np.testing.assert_allclose(gpu["adv"].numpy()[[0, 1, 3]], ref["adv"], rtol=1e-5)
    assert gpu["adv"][2] == 0
    assert gpu["group_offsets"].tolist() == [0, 3, 3]


def test_host_side_errors_enqueue_nothing():
    dev = U.DEV
    f = torch.zeros(4, dtype=torch.float32, device=dev)
    i = torch.zeros(4, dtype=torch.int32, device=dev)
    ws = A.workspace(1 << 16, dev)
    L = A.lib()
    import ctypes
    p = A.Params().c()
    args = lambda ws_ptr, ws_bytes, prm: (f.data_ptr(), i.data_ptr(), i.data_ptr(), i.data_ptr(), 4, 1, 1, 1,
                                          prm, f.data_ptr(), None, None, None, None, None, None, ws_ptr, ws_bytes, None)
    assert L.atgrpo_group_advantages(*args(ws.data_ptr(), 16, ctypes.byref(p))) == A.ERR_WORKSPACE
    assert L.atgrpo_group_advantages(*args(None, 1 << 16, ctypes.byref(p))) == A.ERR_WORKSPACE
    assert L.atgrpo_group_advantages(*args(ws.data_ptr() + 4, 1 << 15, ctypes.byref(p))) == A.ERR_WORKSPACE
    assert L.atgrpo_group_advantages(*args(ws.data_ptr(), 1 << 16, None)) == A.ERR_INVALID_ARG
    bad = A.Params(ddof=3).c()
    assert L.atgrpo_group_advantages(*args(ws.data_ptr(), 1 << 16, ctypes.byref(bad))) == A.ERR_INVALID_ARG


def test_repeatable_bitwise():
    s = WL.make_stress(n_env=2000, n_role=4, n_turn=4, n_tokens=10, seed=9)
    for bucketing in (False, True):
        a = U.gpu_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 2000, 4, 4,
                                   bucketing=bucketing)
        b = U.gpu_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 2000, 4, 4,
                                   bucketing=bucketing)
        for k in a:
            if k != "status":
                assert torch.equal(a[k], b[k]), k


# ------------------------------------------------------------------------------- Eq. 2 reduction
def _gpu_clipped_loss(logp, old_logp, resp, adv, prm=None):
    dev = U.DEV
    prm = prm or A.Params()
    T = logp.numel()
    loss = torch.full((1,), 7.0, dtype=torch.float32, device=dev)
    coef = torch.full((T,), 7.0, dtype=torch.float32, device=dev)
    cc = torch.full((2,), -1, dtype=torch.int64, device=dev)
    status = A.new_status(dev)
    ws = A.workspace(A.atgrpo_clipped_loss_workspace_bytes(T), dev)
    A.atgrpo_clipped_loss(logp.to(dev), old_logp.to(dev), resp.to(dev), adv.to(dev), prm, loss, coef, cc,
                          status, ws)
    torch.cuda.synchronize()
    return loss.cpu(), coef.cpu(), cc.cpu(), int(status.item())


@pytest.mark.parametrize("sigma", [0.05, 0.3])
def test_clipped_loss_vs_oracle(sigma):
    s = WL.make_stress(n_env=500, n_role=4, n_turn=4, n_tokens=300_001, seed=12)
    ref_adv = U.oracle_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], 500, 4, 4)["adv"]
    adv = torch.from_numpy(ref_adv).float()
    old = WL.make_old_logp(s["logp"], 77, sigma)
    old = U.keep_off_the_kinks(s["logp"].numpy(), old)
    loss, coef, cc, status = _gpu_clipped_loss(s["logp"], old, s["resp_of_token"], adv)
    T = s["T"]
    rloss, rcount, rcc = O.policy_loss(s["logp"], old, adv, s["resp_of_token"], np.zeros(T, int), 1)
    assert status == 0
    assert abs(loss.item() - rloss[0]) <= 1e-3 * abs(rloss[0])
    assert cc.tolist() == rcc[0].tolist()
    c = -O.dloss_dlogp(s["logp"], old, adv, s["resp_of_token"], np.zeros(T, int), 1)
    np.testing.assert_allclose(coef.numpy(), c, rtol=2e-5, atol=1e-12)
    if sigma > 0.1:
        assert rcc[0].min() > 1000 and (c == 0).sum() > 1000        # both clip branches exercised


def test_clipped_loss_ratio_one_and_empty():
    g = torch.Generator().manual_seed(1)
    R, T = 100, 5000
    adv = torch.randn(R, generator=g)
    resp = torch.sort(torch.randint(0, R, (T,), generator=g)).values.to(torch.int32)
    logp = -torch.rand(T, generator=g) * 9
    loss, coef, cc, status = _gpu_clipped_loss(logp, logp, resp, adv)
    assert loss.item() == pytest.approx(-adv[resp.long()].double().mean().item(), rel=1e-6)
    assert cc.tolist() == [0, 0]
    z = torch.zeros(0)
    loss, _, cc, _ = _gpu_clipped_loss(z, z, z.to(torch.int32), adv)
    assert loss.item() == 0.0 and cc.tolist() == [0, 0]
