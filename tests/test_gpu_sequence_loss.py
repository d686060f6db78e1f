"""Sequence-level readings of Eq. 2 on the GPU vs. the fp64 oracle -- one ratio per response with the
mean over responses, and the expectation as printed (mean over groups of the per-group mean over
the K candidates): standalone reduction, forward through the LM head, and backward."""
import numpy as np
import pytest
import torch

from oracle import atgrpo_oracle as O
from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu
SEQ = A.Params(reduction=A.REDUCE_SEQUENCE)


def _off_the_sequence_kinks(logp, old, resp, margin=3e-3):
    """Responses whose sequence ratio sits within `margin` of 1 +- eps get ratio 1 instead."""
    resp = np.asarray(resp)
    delta = np.asarray(logp, np.float64) - old.double().numpy()
    out = old.clone()
    for c in np.unique(resp):
        sel = resp == c
        r = np.exp(delta[sel].sum())
        if abs(r - 0.8) < margin or abs(r - 1.2) < margin:
            out[torch.from_numpy(sel)] = torch.from_numpy(np.asarray(logp, np.float32))[torch.from_numpy(sel)]
    return out


def _case(name, sigma):
    b = WL.make_rollout(WL.SPECS[name])
    lse, logp = U.oracle_logprobs(b)
    adv = U.batch_advantages(b)
    old = WL.make_old_logp(torch.from_numpy(logp), b["spec"].seed + 200, sigma)
    old = _off_the_sequence_kinks(logp, old, b["resp_of_token"].numpy())
    return b, lse, logp, adv, old


@pytest.mark.parametrize("name,sigma", [("tiny", 0.03), ("mid_multi", 0.05)])
def test_forward_and_backward_sequence_mode(name, sigma):
    b, lse, logp, adv, old = _case(name, sigma)
    M = b["spec"].n_heads
    head, _, _ = U.oracle_heads(b)
    gl = torch.tensor([1.0, 0.5, 2.0][:M])
    case = U.PolicyCase(b, adv, old, prm=SEQ, grad_loss=gl)
    out = case.fwd()
    assert out["status"] == 0
    rloss, rcount, rcc = O.policy_loss_sequence(logp, old, adv, b["resp_of_token"], head, M)
    np.testing.assert_allclose(out["loss"].numpy(), rloss, rtol=1e-3, atol=1e-7)
    assert np.abs(out["clip_counts"].numpy() - rcc).max() <= 1
    assert rcc.sum() > 0 and rcc.sum() < rcount.sum()            # clipped and unclipped responses both occur
    g = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    assert g["status"] == 0
    dH, dW = O.policy_loss_grads(b["H"], b["W"], b["target"], old, adv, b["resp_of_token"], head,
                                 grad_loss=gl.numpy(), reduction="sequence")
    assert U.rel_fro(g["dH"].numpy(), dH) <= 5e-3
    for m in range(M):
        assert U.rel_fro(g["dW"][m].numpy(), dW[m]) <= 5e-3
    again = case.fwd()
    assert torch.equal(out["loss"], again["loss"])


def test_standalone_sequence_reduction_with_empty_responses():
    s = WL.make_stress(n_env=300, n_role=4, n_turn=4, n_tokens=40_003, seed=31)      # responses of length 0 occur
    R, T = s["R"], s["T"]
    g = torch.Generator().manual_seed(2)
    adv = torch.randn(R, generator=g)
    old = s["logp"] + torch.randn(T, generator=g) * 0.08
    old = _off_the_sequence_kinks(s["logp"].numpy(), old, s["resp_of_token"].numpy())
    dev = U.DEV
    loss = torch.zeros(1, device=dev)
    coef = torch.full((T,), 7.0, device=dev)
    cc = torch.zeros(2, dtype=torch.int64, device=dev)
    st = A.new_status(dev)
    A.atgrpo_clipped_loss(s["logp"].to(dev), old.to(dev), s["resp_of_token"].to(dev), adv.to(dev), SEQ, loss, coef,
                          cc, st, A.workspace(A.atgrpo_clipped_loss_workspace_bytes(T), dev))
    torch.cuda.synchronize()
    head = np.zeros(T, dtype=np.int64)
    rl, rcount, rcc = O.policy_loss_sequence(s["logp"], old, adv, s["resp_of_token"], head, 1)
    assert int(st.item()) == 0
    assert rcount[0] < R                                           # some responses have no token
    assert abs(loss.item() - rl[0]) <= 1e-3 * abs(rl[0])
    assert np.abs(cc.cpu().numpy() - rcc[0]).max() <= 1
    c = -O.dloss_dlogp_sequence(s["logp"], old, adv, s["resp_of_token"], head, 1)
    np.testing.assert_allclose(coef.cpu().numpy(), c, rtol=1e-4, atol=1e-12)


def test_unsorted_tokens_are_flagged():
    dev = U.DEV
    T = 64
    resp = torch.arange(T, dtype=torch.int32) // 8
    resp[20] = 0                                                   # out of order
    z = torch.zeros(T, device=dev)
    st = A.new_status(dev)
    A.atgrpo_clipped_loss(z, z, resp.to(dev), torch.ones(8, device=dev), SEQ, torch.zeros(1, device=dev), None, None,
                          st, A.workspace(A.atgrpo_clipped_loss_workspace_bytes(T), dev))
    torch.cuda.synchronize()
    assert int(st.item()) == A.ERR_BAD_INDEX


# ---------------------------------------------------------------- per-group expectation of Eq. 2
def _group_params(group_of_resp, n_groups):
    dev = U.DEV
    return A.Params(reduction=A.REDUCE_GROUP_MEAN, group_of_resp=group_of_resp.to(torch.int32).to(dev),
                    group_scratch=torch.full((n_groups,), 77, dtype=torch.int32, device=dev))   # stale contents


def test_group_mean_on_groups_of_unequal_size():
    # the stress input: K ~ U{1..16} candidates per group, some responses without tokens
    s = WL.make_stress(n_env=300, n_role=4, n_turn=4, n_tokens=40_003, seed=33, shuffle=False)
    R, T, G = s["R"], s["T"], s["G"]
    key = O.group_key(s["env_id"], s["role_id"], s["turn_id"], s["n_env"], s["n_role"], s["n_turn"])
    g = torch.Generator().manual_seed(3)
    adv = torch.randn(R, generator=g)
    old = s["logp"] + torch.randn(T, generator=g) * 0.08
    old = _off_the_sequence_kinks(s["logp"].numpy(), old, s["resp_of_token"].numpy())
    dev = U.DEV
    prm = _group_params(torch.from_numpy(key), G)
    loss = torch.zeros(1, device=dev)
    coef = torch.full((T,), 7.0, device=dev)
    cc = torch.zeros(2, dtype=torch.int64, device=dev)
    st = A.new_status(dev)
    ws = A.workspace(A.atgrpo_clipped_loss_workspace_bytes(T), dev)
    args = (s["logp"].to(dev), old.to(dev), s["resp_of_token"].to(dev), adv.to(dev), prm, loss, coef, cc, st, ws)
    A.atgrpo_clipped_loss(*args)
    torch.cuda.synchronize()
    head = np.zeros(T, dtype=np.int64)
    rl, rcount, rcc = O.policy_loss_sequence(s["logp"], old, adv, s["resp_of_token"], head, 1, group_of_resp=key)
    per_resp, n_resp_present, _ = O.policy_loss_sequence(s["logp"], old, adv, s["resp_of_token"], head, 1)
    assert int(st.item()) == 0
    assert rcount[0] < n_resp_present[0] and abs(rl[0] - per_resp[0]) > 1e-3 * abs(rl[0])   # the two means differ here
    assert abs(loss.item() - rl[0]) <= 1e-3 * abs(rl[0])
    assert np.abs(cc.cpu().numpy() - rcc[0]).max() <= 1
    c = -O.dloss_dlogp_sequence(s["logp"], old, adv, s["resp_of_token"], head, 1, group_of_resp=key)
    np.testing.assert_allclose(coef.cpu().numpy(), c, rtol=1e-4, atol=1e-12)
    first = loss.clone()
    A.atgrpo_clipped_loss(*args)                                   # the scratch now holds the last call's counts
    torch.cuda.synchronize()
    assert torch.equal(first, loss)


def test_group_mean_through_the_lm_head():
    b, lse, logp, adv, old = _case("mid_multi", 0.05)
    spec = b["spec"]
    key = O.group_key(b["env_id"], b["role_id"], b["turn_id"], spec.n_env, spec.n_role, spec.n_turn)
    G = spec.n_env * spec.n_role * spec.n_turn
    M = spec.n_heads
    head, _, _ = U.oracle_heads(b)
    gl = torch.tensor([1.0, 0.5, 2.0][:M])
    # unequal weights come from responses that share a group with fewer present members: keep all
    # tokens (the GEMM inputs stay as generated) but move one response of each even group to a
    # group of its own, which changes K_g without touching any token
    key2 = key.copy()
    moved = 0
    for q in range(0, G, 2):
        members = np.nonzero(key == q)[0]
        spare = (q + 1) if (q + 1) < G and (q + 1) % 2 == 1 else None
        if spare is not None and members.size > 1 and \
                b["role_id"][members[0]] == b["role_id"][np.nonzero(key == spare)[0][0]]:
            key2[members[0]] = spare
            moved += 1
    assert moved > 0
    prm = _group_params(torch.from_numpy(key2), G)
    case = U.PolicyCase(b, adv, old, prm=prm, grad_loss=gl)
    out = case.fwd()
    assert out["status"] == 0
    rloss, _, _ = O.policy_loss_sequence(logp, old, adv, b["resp_of_token"], head, M, group_of_resp=key2)
    np.testing.assert_allclose(out["loss"].numpy(), rloss, rtol=1e-3, atol=1e-7)
    g = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    assert g["status"] == 0
    dH, dW = O.policy_loss_grads(b["H"], b["W"], b["target"], old, adv, b["resp_of_token"], head,
                                 grad_loss=gl.numpy(), reduction="sequence", group_of_resp=key2)
    assert U.rel_fro(g["dH"].numpy(), dH) <= 5e-3
    for m in range(M):
        assert U.rel_fro(g["dW"][m].numpy(), dW[m]) <= 5e-3


def test_group_mean_flags_a_bad_group_id():
    dev = U.DEV
    T, R = 64, 8
    resp = torch.arange(T, dtype=torch.int32) // 8
    group = torch.tensor([0, 0, 1, 1, 9, 2, 2, 2])                 # response 4: group out of range
    prm = _group_params(group, 3)
    lp = torch.zeros(T, device=dev)
    adv = torch.arange(1, R + 1, dtype=torch.float32)
    loss = torch.zeros(1, device=dev)
    st = A.new_status(dev)
    A.atgrpo_clipped_loss(lp, lp, resp.to(dev), adv.to(dev), prm, loss, None, None, st,
                          A.workspace(A.atgrpo_clipped_loss_workspace_bytes(T), dev))
    torch.cuda.synchronize()
    assert int(st.item()) == A.ERR_BAD_INDEX
    # the response is left out: three groups remain, ratio 1, term = A
    assert loss.item() == pytest.approx(-((1 + 2) / 2 + (3 + 4) / 2 + (6 + 7 + 8) / 3) / 3, rel=1e-6)
