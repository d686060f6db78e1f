"""Kept logits (params.logits): the forward call stores z = H W_m^T, the backward call reads it back
instead of repeating the contraction.  The stored logits are checked against the oracle's fp64
logits; the gradients against the oracle and, bit for bit, against the recomputing backward."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import atgrpo_oracle as O
from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu

# several vocabulary chunks at a small d, three heads; and a vocabulary that is no multiple of 8
WIDE = WL.RolloutSpec("kept_wide", 6, 3, 2, 4, (24, 8, 8), (40, 24, 24), 64, 151936, 3, 1261)
RAGGED = WL.RolloutSpec("kept_ragged", 5, 2, 2, 4, (8, 8), (40, 40), 128, 2048 + 517, 1, 1262)


def _lend(case, T, V):
    """A logits buffer full of NaN: whatever the library does not write must never be used."""
    ld = (V + 255) // 256 * 256
    assert A.atgrpo_policy_loss_logits_bytes(T, V) == T * ld * 4
    assert A.atgrpo_policy_loss_logits_bytes(T, V, A.LOGITS_Q16) == T * ld * 2 + T * (ld // 32) * 4
    return case.lend_logits(), ld


def _case(spec, prm=None, zero_every=5):
    b = WL.make_rollout(spec)
    adv = torch.where(torch.arange(b["R"]) % zero_every == 0, 0.0, 1.0) * (torch.arange(b["R"]) % 7 - 3.0)
    case = U.PolicyCase(b, adv, torch.zeros(b["T"]), prm=prm)
    f = case.fwd(want_routing=False)
    assert f["status"] == 0
    case.old_logp = (f["logp"] + 0.3 * torch.sin(torch.arange(b["T"]).float())).to(U.DEV)
    return b, case, f


@pytest.mark.parametrize("name", ["mid", "mid_multi"])
def test_forward_stores_the_logits_of_every_routed_token(name):
    spec = WL.SPECS[name]
    b = WL.make_rollout(spec)
    if spec.n_heads > 1:
        b["role_of_token"][7] = spec.n_role + 3            # one token that belongs to no policy
    T, V, M = b["T"], spec.V, spec.n_heads
    adv = torch.ones(b["R"])
    adv[::3] = 0.0                                         # every third response carries no gradient
    case = U.PolicyCase(b, adv, torch.zeros(T))
    plain = case.fwd(want_routing=False)
    buf, ld = _lend(case, T, V)
    kept = case.fwd(want_routing=False)
    assert kept["status"] == plain["status"]
    # lending the buffer changes nothing else (the unroutable token's entries are left untouched, 7.0)
    for k in ("loss", "logp", "lse", "clip_counts"):
        assert torch.equal(kept[k], plain[k]), k
    z = buf.view(T, ld)[:, :V].cpu().double().numpy()
    head = np.zeros(T, dtype=np.int64)
    if spec.n_heads > 1:
        role = b["role_of_token"].numpy()
        ok = (role >= 0) & (role < spec.n_role)
        head = np.where(ok, b["head_of_role"].numpy()[np.clip(role, 0, spec.n_role - 1)], -1)
    live = adv.numpy()[b["resp_of_token"].numpy()] != 0
    assert 0 < live.sum() < T
    Hf = b["H"].double().numpy()
    for m in range(M):
        rows = np.nonzero((head == m) & live)[0]
        ref = Hf[rows] @ b["W"][m].double().numpy().T
        # bf16 x bf16 products are exact in fp32; only the order of the d additions differs
        np.testing.assert_allclose(z[rows], ref, rtol=0, atol=2e-5 * np.sqrt(spec.d) * np.abs(ref).max())
    lost = np.nonzero((head < 0) | ~live)[0]
    assert np.isnan(z[lost]).all()         # rows of unroutable tokens and of zero-advantage responses are not written
    assert (head < 0).sum() == (1 if spec.n_heads > 1 else 0)


@pytest.mark.parametrize("spec,prm", [
    (WL.SPECS["mid"], A.Params()),
    (WL.SPECS["mid_multi"], A.Params(dH_dtype=A.F32, dW_dtype=A.BF16)),
    (RAGGED, A.Params(reduction=A.REDUCE_SEQUENCE)),
    (WIDE, A.Params()),
], ids=["mid", "mid_multi_f32_bf16", "ragged_sequence", "wide_three_chunks"])
def test_backward_from_kept_logits_equals_the_recomputing_backward_bit_for_bit(spec, prm):
    b, case, f = _case(spec, prm)
    T, d, V, M = b["T"], spec.d, spec.V, spec.n_heads
    if spec is WIDE:
        assert A.atgrpo_policy_loss_bwd_chunks(T, d, V, M)[0] >= 2
    ref = case.bwd(f["logp"], f["lse"])
    assert ref["status"] == 0
    buf, ld = _lend(case, T, V)
    f2 = case.fwd(want_routing=False)
    assert f2["status"] == 0 and torch.equal(f2["logp"], f["logp"]) and torch.equal(f2["lse"], f["lse"])
    got = case.bwd(f["logp"], f["lse"])
    assert got["status"] == 0
    assert torch.equal(got["dH"], ref["dH"])
    for m in range(M):
        assert torch.equal(got["dW"][m], ref["dW"][m]), m
    assert any(float(w.abs().max()) > 0 for w in got["dW"])


def test_backward_from_kept_logits_matches_the_oracle():
    spec = WL.SPECS["mid_multi"]
    b = WL.make_rollout(spec)
    T, V, M = b["T"], spec.V, spec.n_heads
    lse, logp = U.oracle_logprobs(b)
    adv = U.batch_advantages(b)
    old = U.keep_off_the_kinks(logp, WL.make_old_logp(torch.from_numpy(logp), 23, 0.3))
    head, _, _ = U.oracle_heads(b)
    gl = torch.tensor([0.5, 1.0, 2.0])
    case = U.PolicyCase(b, adv, old, prm=A.Params(dH_dtype=A.F32), grad_loss=gl)
    _lend(case, T, V)
    f = case.fwd()
    assert f["status"] == 0
    g = case.bwd(f["logp"], f["lse"])
    assert g["status"] == 0
    dH, dW = O.policy_loss_grads(b["H"], b["W"], b["target"], old, adv, b["resp_of_token"], head,
                                 grad_loss=gl.numpy())
    U.check_rows(g["dH"].numpy(), dH, "dH")
    for m in range(M):
        U.check_rows(g["dW"][m].numpy(), dW[m], "dW[%d]" % m)


def test_accumulation_and_notification_work_from_kept_logits():
    b, case, f = _case(WIDE, A.Params(accumulate_dW=1))
    T, d, V, M = b["T"], WIDE.d, WIDE.V, WIDE.n_heads
    once = case.bwd(f["logp"], f["lse"])                    # dW starts at zero when accumulating
    buf, _ = _lend(case, T, V)
    assert case.fwd(want_routing=False)["status"] == 0
    n_chunks, _ = A.atgrpo_policy_loss_bwd_chunks(T, d, V, M)
    events = [torch.cuda.Event() for _ in range(n_chunks)]
    dH = torch.full((T, d), 7.0, dtype=torch.bfloat16, device=U.DEV)
    dW = [torch.zeros((V, d), dtype=torch.float32, device=U.DEV) for _ in range(M)]
    status = A.new_status(U.DEV)
    ws = A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, d, V, M, True), U.DEV)
    for _ in range(2):
        A.atgrpo_policy_loss_bwd(case.H, case.W, case.target, case.role_of_token, case.head_of_role,
                                 case.resp_of_token, case.adv, case.old_logp, f["logp"].to(U.DEV),
                                 f["lse"].to(U.DEV), None, case.prm, dH, dW, device_status=status, workspace=ws,
                                 chunk_events=events)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and all(ev.query() for ev in events)
    assert torch.equal(dH.float().cpu(), once["dH"])
    for m in range(M):
        assert torch.equal(dW[m].cpu(), once["dW"][m] + once["dW"][m])


def test_a_logits_buffer_that_is_too_small_or_misaligned_is_rejected():
    spec = WL.SPECS["tiny"]
    b = WL.make_rollout(spec)
    T, V = b["T"], spec.V
    case = U.PolicyCase(b, torch.ones(b["R"]), torch.zeros(T))
    n = A.atgrpo_policy_loss_logits_bytes(T, V) // 4
    big = torch.zeros(n + 64, dtype=torch.float32, device=U.DEV)
    for bad in (big[: n - 1], big[1: n + 1]):
        case.prm = dataclasses.replace(case.prm, logits=bad)
        with pytest.raises(A.AtgrpoError):
            case.fwd(want_routing=False)
        with pytest.raises(A.AtgrpoError):
            case.bwd(torch.zeros(T), torch.zeros(T))
    assert A.atgrpo_policy_loss_logits_bytes(0, V) == 0
    case.prm = dataclasses.replace(case.prm, logits=big[:n])
    assert case.fwd(want_routing=False)["status"] == 0


def test_bad_target_with_kept_logits_is_flagged_in_both_calls_and_stays_in_bounds():
    # a target id outside the vocabulary is read as token 0 (documented); forward and backward each flag it
    b, case, f = _case(WL.SPECS["tiny"])
    T, V = b["T"], WL.SPECS["tiny"].V
    j = int((b["resp_of_token"] == 1).nonzero()[0])        # a token whose response has a non-zero advantage
    b2 = dict(b)
    b2["target"] = b["target"].clone()
    b2["target"][j] = V + 5
    b0 = dict(b)
    b0["target"] = b["target"].clone()
    b0["target"][j] = 0
    adv = case.adv.cpu()
    res = []
    for batch in (b2, b0):
        c = U.PolicyCase(batch, adv, torch.zeros(T))
        c.lend_logits()
        out = c.fwd(want_routing=False)
        c.old_logp = (out["logp"] + 0.1).to(U.DEV)
        g = c.bwd(out["logp"], out["lse"])
        res.append((out, g))
    (o_bad, g_bad), (o_ok, g_ok) = res
    assert o_bad["status"] == A.ERR_BAD_INDEX and g_bad["status"] == A.ERR_BAD_INDEX
    assert o_ok["status"] == 0 and g_ok["status"] == 0
    assert torch.equal(o_bad["logp"], o_ok["logp"]) and torch.equal(g_bad["dH"], g_ok["dH"])
    assert torch.equal(g_bad["dW"][0], g_ok["dW"][0])


def test_group_mean_reduction_from_kept_logits():
    # the per-group reading of Eq. 2 changes only the gradient factor: kept and recomputed logits agree bit for bit
    spec = WL.SPECS["mid_multi"]
    b = WL.make_rollout(spec)
    T, V, M = b["T"], spec.V, spec.n_heads
    ref = U.oracle_group_advantages(b["rewards"], b["env_id"], b["role_id"], b["turn_id"], spec.n_env, spec.n_role,
                                    spec.n_turn)
    G = spec.n_env * spec.n_role * spec.n_turn
    gof = torch.from_numpy(ref["group_of_cand"].astype(np.int32)).to(U.DEV)
    prm = A.Params(reduction=A.REDUCE_GROUP_MEAN, group_of_resp=gof,
                   group_scratch=torch.zeros(G, dtype=torch.int32, device=U.DEV))
    case = U.PolicyCase(b, torch.from_numpy(ref["adv"]), torch.zeros(T), prm=prm)
    f = case.fwd(want_routing=False)
    assert f["status"] == 0
    case.old_logp = (f["logp"] + 0.002 * torch.sin(torch.arange(T).float())).to(U.DEV)
    case.lend_logits()
    assert case.fwd(want_routing=False)["status"] == 0
    g = case.bwd_both_ways(f["logp"], f["lse"])
    assert g["status"] == 0 and float(g["dH"].abs().max()) > 0


# ------------------------------------------------------------------ the compact format (16-bit codes)

@pytest.mark.parametrize("name", ["mid", "mid_multi"])
def test_codes_decode_to_the_oracle_logits_within_half_a_step(name):
    spec = WL.SPECS[name]
    b = WL.make_rollout(spec)
    T, V, M = b["T"], spec.V, spec.n_heads
    adv = torch.ones(b["R"])
    adv[::4] = 0.0
    case = U.PolicyCase(b, adv, torch.zeros(T))
    plain = case.fwd(want_routing=False)
    buf = case.lend_logits(A.LOGITS_Q16)
    kept = case.fwd(want_routing=False)
    for k in ("loss", "logp", "lse", "clip_counts"):
        assert torch.equal(kept[k], plain[k]), k
    ld = (V + 255) // 256 * 256
    raw = buf.cpu().numpy()
    codes = raw[: T * ld * 2].view(np.uint16).reshape(T, ld).astype(np.float64)
    refs = raw[T * ld * 2:].view(np.float32).reshape(T, ld // 32).astype(np.float64)
    z = (np.repeat(refs, 32, axis=1) - codes / 1024.0)[:, :V]
    head, _, _ = U.oracle_heads(b)
    live = adv.numpy()[b["resp_of_token"].numpy()] != 0
    Hf = b["H"].double().numpy()
    for m in range(M):
        rows = np.nonzero((head == m) & live)[0]
        ref = Hf[rows] @ b["W"][m].double().numpy().T
        # the block maximum is the fp32 logit itself; every other logit is at most half a code step off it
        blockmax = np.stack([ref[:, c:c + 32].max(axis=1) for c in range(0, V, 32)], axis=1)
        np.testing.assert_allclose(refs[rows][:, : blockmax.shape[1]], blockmax, rtol=0, atol=1e-4)
        assert np.abs(z[rows] - ref).max() <= 2.0 ** -11 + 1e-4
        assert (codes[rows][:, :V].min(axis=1) == 0).all()          # the maximum of a block has code 0
    dead = np.nonzero(~live)[0]
    assert (raw[: T * ld * 2].view(np.uint16).reshape(T, ld)[dead] == 0xFFFF).all()    # rows that are not kept stay untouched


@pytest.mark.parametrize("spec,prm", [
    (WL.SPECS["mid"], A.Params()),
    (WL.SPECS["mid_multi"], A.Params(dH_dtype=A.F32, dW_dtype=A.BF16)),
    (RAGGED, A.Params(reduction=A.REDUCE_SEQUENCE)),
    (WIDE, A.Params()),
], ids=["mid", "mid_multi_f32_bf16", "ragged_sequence", "wide_three_chunks"])
def test_backward_from_codes_stays_close_to_the_recomputing_backward(spec, prm):
    b, case, f = _case(spec, prm)
    T, d, V, M = b["T"], spec.d, spec.V, spec.n_heads
    ref = case.bwd(f["logp"], f["lse"])
    case.lend_logits(A.LOGITS_Q16)
    f2 = case.fwd(want_routing=False)
    assert f2["status"] == 0 and torch.equal(f2["logp"], f["logp"])
    got = case.bwd(f["logp"], f["lse"])
    assert got["status"] == 0
    # |dz - dz~| <= 4.9e-4 * p elementwise before the bf16 rounding both ways share: the results differ by far
    # less than either differs from the exact gradient (5e-3 is the tolerance against the oracle)
    assert U.rel_fro(got["dH"].numpy(), ref["dH"].numpy()) <= 1.5e-3
    for m in range(M):
        if float(ref["dW"][m].abs().max()) > 0:
            assert U.rel_fro(got["dW"][m].numpy(), ref["dW"][m].numpy()) <= 1.5e-3, m
        else:
            assert (got["dW"][m] == 0).all()
    assert (got["dH"][ref["dH"].abs().sum(1) == 0] == 0).all()     # rows without a gradient stay exactly zero


def test_backward_from_codes_matches_the_oracle():
    spec = WL.SPECS["mid_multi"]
    b = WL.make_rollout(spec)
    T, V, M = b["T"], spec.V, spec.n_heads
    lse, logp = U.oracle_logprobs(b)
    adv = U.batch_advantages(b)
    old = U.keep_off_the_kinks(logp, WL.make_old_logp(torch.from_numpy(logp), 23, 0.3))
    head, _, _ = U.oracle_heads(b)
    gl = torch.tensor([0.5, 1.0, 2.0])
    case = U.PolicyCase(b, adv, old, prm=A.Params(dH_dtype=A.F32), grad_loss=gl)
    case.lend_logits(A.LOGITS_Q16)
    f = case.fwd()
    assert f["status"] == 0
    g = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    assert g["status"] == 0
    dH, dW = O.policy_loss_grads(b["H"], b["W"], b["target"], old, adv, b["resp_of_token"], head,
                                 grad_loss=gl.numpy())
    U.check_rows(g["dH"].numpy(), dH, "dH")
    for m in range(M):
        U.check_rows(g["dW"][m].numpy(), dW[m], "dW[%d]" % m)


def test_a_code_buffer_that_is_too_small_or_an_unknown_format_is_rejected():
    spec = WL.SPECS["tiny"]
    b = WL.make_rollout(spec)
    T, V = b["T"], spec.V
    case = U.PolicyCase(b, torch.ones(b["R"]), torch.zeros(T))
    n = A.atgrpo_policy_loss_logits_bytes(T, V, A.LOGITS_Q16)
    big = torch.zeros(n, dtype=torch.uint8, device=U.DEV)
    case.prm = dataclasses.replace(case.prm, logits=big[: n - 4], logits_format=A.LOGITS_Q16)
    with pytest.raises(A.AtgrpoError):
        case.fwd(want_routing=False)
    case.prm = dataclasses.replace(case.prm, logits=big, logits_format=7)
    with pytest.raises(A.AtgrpoError):
        case.fwd(want_routing=False)
    assert A.atgrpo_policy_loss_logits_bytes(T, V, 7) == 0
    case.prm = dataclasses.replace(case.prm, logits=big, logits_format=A.LOGITS_Q16)
    assert case.fwd(want_routing=False)["status"] == 0
