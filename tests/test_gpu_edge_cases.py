"""Degenerate and extreme shapes of the policy loss through the C ABI: tiny vocabulary, minimal d,
a single token, the maximum number of heads with empty ones, T = 0, strided H."""
import numpy as np
import pytest
import torch

from oracle import atgrpo_oracle as O
from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu


def _check(b, sigma=0.3, prm=None, tol_fro=5e-3):
    lse, logp = U.oracle_logprobs(b)
    adv = U.batch_advantages(b)
    old = U.keep_off_the_kinks(logp, WL.make_old_logp(torch.from_numpy(logp), 11, sigma))
    head, offsets, perm = U.oracle_heads(b)
    M = b["spec"].n_heads
    case = U.PolicyCase(b, adv, old, prm=prm)
    out = case.fwd()
    assert out["status"] == 0
    assert np.array_equal(out["role_offsets"].numpy(), offsets) and np.array_equal(out["role_perm"].numpy(), perm)
    assert np.abs(out["logp"].numpy() - logp).max() <= 1e-3
    assert np.abs(out["lse"].numpy() - lse).max() <= 1e-3
    rl, _, _ = O.policy_loss(logp, old, adv, b["resp_of_token"], head, M)
    np.testing.assert_allclose(out["loss"].numpy(), rl, rtol=1e-3, atol=1e-7)
    g = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    assert g["status"] == 0
    dH, dW = O.policy_loss_grads(b["H"], b["W"], b["target"], old, adv, b["resp_of_token"], head)
    if np.linalg.norm(dH) > 0:
        assert U.rel_fro(g["dH"].numpy(), dH) <= tol_fro
    for m in range(M):
        if np.linalg.norm(dW[m]) > 0:
            assert U.rel_fro(g["dW"][m].numpy(), dW[m]) <= tol_fro
        else:
            assert (g["dW"][m] == 0).all()
    # once more with the logits kept by the forward: same forward outputs, same gradient bits
    case.lend_logits()
    out2 = case.fwd()
    assert out2["status"] == 0
    for k in ("loss", "logp", "lse", "role_offsets", "role_perm", "clip_counts"):
        assert torch.equal(out2[k], out[k]), k
    g2 = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    assert g2["status"] == 0 and torch.equal(g2["dH"], g["dH"])
    for m in range(M):
        assert torch.equal(g2["dW"][m], g["dW"][m]), m
    # and with the logits kept as 16-bit codes: the oracle's tolerances again
    case.lend_logits(A.LOGITS_Q16)
    out3 = case.fwd()
    assert out3["status"] == 0 and torch.equal(out3["logp"], out["logp"]) and torch.equal(out3["lse"], out["lse"])
    g3 = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    assert g3["status"] == 0
    if np.linalg.norm(dH) > 0:
        assert U.rel_fro(g3["dH"].numpy(), dH) <= tol_fro
    for m in range(M):
        if np.linalg.norm(dW[m]) > 0:
            assert U.rel_fro(g3["dW"][m].numpy(), dW[m]) <= tol_fro
        else:
            assert (g3["dW"][m] == 0).all()
    return out, g


def test_vocabulary_smaller_than_one_tile_and_minimal_d():
    _check(WL.make_rollout(WL.RolloutSpec("v100", 2, 2, 1, 4, (5, 5), (30, 30), 64, 100, 1, 501, 0)))
    _check(WL.make_rollout(WL.RolloutSpec("v257", 2, 2, 1, 4, (5, 5), (30, 30), 72, 257, 1, 502, 0)))


def test_d_not_a_multiple_of_the_k_step_or_the_column_tile():
    # d = 328: 5.125 k-steps of 64, 1.28 column tiles of 256 (zero-filled by TMA, masked on store)
    _check(WL.make_rollout(WL.RolloutSpec("d328", 3, 2, 2, 4, (10, 10), (50, 50), 328, 1000, 1, 503, 1)))


def test_eight_heads_with_empty_ones():
    spec = WL.RolloutSpec("m8", 3, 8, 1, 4, (3,) * 8, (20,) * 8, 128, 700, 8, 504, 1)
    b = WL.make_rollout(spec)
    b["head_of_role"] = torch.tensor([7, 0, 7, 3, 3, 0, 5, 5], dtype=torch.int32)   # heads 1, 2, 4, 6 unused
    out, g = _check(b)
    for m in (1, 2, 4, 6):
        assert out["loss"][m] == 0 and (g["dW"][m] == 0).all()


def test_single_token_and_single_response():
    spec = WL.RolloutSpec("one", 1, 1, 1, 2, (1,), (1,), 64, 300, 1, 505, 0)
    _check(WL.make_rollout(spec))


def test_zero_tokens():
    dev = U.DEV
    d, V = 64, 512
    W = [torch.zeros(V, d, dtype=torch.bfloat16, device=dev)]
    H = torch.zeros(0, d, dtype=torch.bfloat16, device=dev)
    e_i = torch.zeros(0, dtype=torch.int32, device=dev)
    e_f = torch.zeros(0, dtype=torch.float32, device=dev)
    adv = torch.zeros(4, device=dev)
    loss = torch.full((1,), 7.0, device=dev)
    st = A.new_status(dev)
    ws = A.workspace(A.atgrpo_policy_loss_workspace_bytes(0, d, V, 1, True), dev)
    A.atgrpo_policy_loss_fwd(H, W, e_i, None, None, e_i, adv, e_f, A.Params(), loss, e_f, e_f, device_status=st, workspace=ws)
    dW = [torch.full((V, d), 7.0, device=dev)]
    A.atgrpo_policy_loss_bwd(H, W, e_i, None, None, e_i, adv, e_f, e_f, e_f, None, A.Params(), H, dW, st, ws)
    torch.cuda.synchronize()
    assert loss.item() == 0 and (dW[0] == 0).all() and int(st.item()) == 0
    # the same with a (necessarily empty) logits buffer lent
    assert A.atgrpo_policy_loss_logits_bytes(0, V) == 0
    prm = A.Params(logits=torch.zeros(64, device=dev))
    loss.fill_(7.0), dW[0].fill_(7.0)
    A.atgrpo_policy_loss_fwd(H, W, e_i, None, None, e_i, adv, e_f, prm, loss, e_f, e_f, device_status=st, workspace=ws)
    A.atgrpo_policy_loss_bwd(H, W, e_i, None, None, e_i, adv, e_f, e_f, e_f, None, prm, H, dW, st, ws)
    torch.cuda.synchronize()
    assert loss.item() == 0 and (dW[0] == 0).all() and int(st.item()) == 0


def test_strided_hidden_states():
    # H as a column slice of a wider activation buffer: row stride ldH > d
    b = WL.make_rollout(WL.SPECS["tiny"])
    lse, logp = U.oracle_logprobs(b)
    dev = U.DEV
    T, d = b["H"].shape
    wide = torch.zeros(T, d + 64, dtype=torch.bfloat16, device=dev)
    wide[:, :d] = b["H"].to(dev)
    Hs = wide[:, :d]
    assert Hs.stride(0) == d + 64
    f32 = torch.float32
    loss, lp, ls = torch.zeros(1, device=dev), torch.zeros(T, device=dev), torch.zeros(T, device=dev)
    adv = torch.zeros(b["R"], device=dev)
    ws = A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, d, b["spec"].V, 1, False), dev)
    st = A.new_status(dev)
    import ctypes
    W = [b["W"][0].to(dev)]
    target, resp, old = b["target"].to(dev), b["resp_of_token"].to(dev), torch.zeros(T, device=dev)
    prm = A.Params().c()
    rc = A.lib().atgrpo_policy_loss_fwd(
        Hs.data_ptr(), Hs.stride(0), A._ptr_array(W, torch.bfloat16), 1, target.data_ptr(), None, None, 0,
        resp.data_ptr(), adv.data_ptr(), b["R"], old.data_ptr(), T, d, b["spec"].V, ctypes.byref(prm),
        loss.data_ptr(), lp.data_ptr(), ls.data_ptr(), None, None, None, st.data_ptr(), ws.data_ptr(), ws.numel(),
        None)
    assert rc == A.OK
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert np.abs(lp.cpu().numpy() - logp).max() <= 1e-3


@pytest.mark.parametrize("seed", range(8))
def test_random_shapes(seed):
    """Seeded random shapes: d any multiple of 8, V anywhere around the tile sizes, 1-4 heads, short and
    long responses, both reductions -- forward, backward and routing against the oracle."""
    g = np.random.default_rng(1000 + seed)
    n_role = int(g.integers(1, 5))
    heads = n_role if g.random() < 0.6 else 1
    d = int(g.integers(8, 65)) * 8                                  # 64 .. 512
    V = int(g.choice([int(g.integers(1, 300)), int(g.integers(300, 3000)), 256, 512, 1024 + int(g.integers(0, 3))]))
    lo = tuple(int(x) for x in g.integers(1, 20, n_role))
    hi = tuple(int(l + g.integers(0, 120)) for l in lo)
    spec = WL.RolloutSpec(f"rnd{seed}", int(g.integers(1, 5)), n_role, int(g.integers(1, 4)), int(g.integers(1, 6)),
                          lo, hi, d, V, heads, 7000 + seed, 1)
    b = WL.make_rollout(spec)
    _check(b, sigma=0.3)
    if seed % 2 == 0:                                               # sequence-level reduction on half of them
        lse, logp = U.oracle_logprobs(b)
        adv = U.batch_advantages(b)
        old = WL.make_old_logp(torch.from_numpy(logp), 13, 0.02)
        head, _, _ = U.oracle_heads(b)
        resp = b["resp_of_token"].numpy()
        delta = logp - old.double().numpy()
        for c in np.unique(resp):                                   # keep sequence ratios off the kinks
            r = np.exp(delta[resp == c].sum())
            if abs(r - 0.8) < 3e-3 or abs(r - 1.2) < 3e-3:
                old[torch.from_numpy(resp == c)] = torch.from_numpy(logp).float()[torch.from_numpy(resp == c)]
        prm = A.Params(reduction=A.REDUCE_SEQUENCE)
        case = U.PolicyCase(b, adv, old, prm=prm)
        out = case.fwd()
        rl, _, _ = O.policy_loss_sequence(logp, old, adv, b["resp_of_token"], head, heads)
        np.testing.assert_allclose(out["loss"].numpy(), rl, rtol=1e-3, atol=1e-7)
        gr = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
        dH, dW = O.policy_loss_grads(b["H"], b["W"], b["target"], old, adv, b["resp_of_token"], head,
                                     reduction="sequence")
        if np.linalg.norm(dH) > 0:
            assert U.rel_fro(gr["dH"].numpy(), dH) <= 5e-3
        for m in range(heads):
            if np.linalg.norm(dW[m]) > 0:
                assert U.rel_fro(gr["dW"][m].numpy(), dW[m]) <= 5e-3


def test_all_advantages_zero_gives_zero_gradients():
    # every group ties: no token carries a gradient, the backward GEMMs get no rows at all
    b = WL.make_rollout(WL.SPECS["mid_multi"])
    adv = torch.zeros(b["R"], dtype=torch.float64)
    lse, logp = U.oracle_logprobs(b)
    old = WL.make_old_logp(torch.from_numpy(logp), 3, 0.3)
    case = U.PolicyCase(b, adv, old)
    out = case.fwd()
    assert (out["loss"] == 0).all() and out["status"] == 0
    g = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    assert g["status"] == 0 and (g["dH"] == 0).all()
    for w in g["dW"]:
        assert (w == 0).all()


def test_a_bounded_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    # A tiny library kernel waits on a barrier nothing arrives on, with a 2 ms limit: both kinds of
    # wait (spinning and backing off) must give up, the status word must say so, and the next
    # regular call on the same stream must work and match the oracle.
    dev = U.DEV
    st = A.new_status(dev)
    waited = torch.zeros(2, dtype=torch.int32, device=dev)
    assert A.atgrpo_selftest_bounded_wait(2_000_000, st, waited) == A.OK
    torch.cuda.synchronize()
    assert int(st.item()) == A.ERR_TIMEOUT
    assert waited.cpu().tolist() == [1, 1]
    assert A.atgrpo_selftest_bounded_wait(10**9, st, waited) == A.ERR_INVALID_ARG     # limits are capped
    _check(WL.make_rollout(WL.SPECS["tiny"]))


@pytest.mark.parametrize("scale", [6.0, 16.0])
def test_peaked_distributions_with_logits_tens_of_units_apart(scale):
    # hidden states scaled up: logits of std 6 / 16 (extremes beyond +-25 / +-70), softmax concentrated on a few
    # entries, most probabilities underflowing; all three ways of obtaining the logits in the backward
    spec = WL.RolloutSpec("peaked", 4, 2, 2, 4, (10, 10), (40, 40), 256, 5000 + 37, 2, 611, 1)
    b = WL.make_rollout(spec)
    b["H"] = (b["H"].float() * scale).to(torch.bfloat16)
    _check(b, sigma=0.3)
