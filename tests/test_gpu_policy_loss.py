"""CUDA policy loss through the LM head (forward and backward) vs. the fp64 oracle, element by
element on shapes that span several tiles and ragged tails, through the C ABI.
Tolerances (bf16 operands, fp32 accumulation; oracle on the same bf16-rounded inputs):
token log-probs <= 1e-3 absolute, loss <= 1e-3 relative, dH and dW <= 5e-3 relative Frobenius;
routing bit-exact.  The gradients are also held to a per-row bound (U.check_rows), so one wrong
token or vocabulary row cannot hide inside the norm of the whole tensor."""
import numpy as np
import pytest
import torch

from oracle import atgrpo_oracle as O
from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu

_cache = {}


def _case(name, sigma=0.05):
    """Batch + oracle log-probs + advantages + old_logp (built from the ORACLE's logp)."""
    key = (name, sigma)
    if key not in _cache:
        b = WL.make_rollout(WL.SPECS[name])
        lse, logp = U.oracle_logprobs(b)
        adv = U.batch_advantages(b)
        old = WL.make_old_logp(torch.from_numpy(logp), b["spec"].seed + 100, sigma)
        old = U.keep_off_the_kinks(logp, old)
        _cache[key] = (b, lse, logp, adv, old)
    return _cache[key]


@pytest.mark.parametrize("name", ["tiny", "mid", "mid_multi"])
@pytest.mark.parametrize("sigma", [0.05, 0.3])
def test_forward(name, sigma):
    b, lse, logp, adv, old = _case(name, sigma)
    case = U.PolicyCase(b, adv, old)
    out = case.fwd()
    assert out["status"] == 0
    head, offsets, perm = U.oracle_heads(b)
    assert np.array_equal(out["role_offsets"].numpy(), offsets)            # bit-exact routing
    assert np.array_equal(out["role_perm"].numpy(), perm)
    assert np.abs(out["lse"].numpy() - lse).max() <= 1e-3
    assert np.abs(out["logp"].numpy() - logp).max() <= 1e-3
    rloss, rcount, rcc = O.policy_loss(logp, old, adv, b["resp_of_token"], head, case.M)
    np.testing.assert_allclose(out["loss"].numpy(), rloss, rtol=1e-3)
    # a clip count may differ only for tokens whose ratio is within rounding of a boundary
    assert np.abs(out["clip_counts"].numpy() - rcc).max() <= 2
    again = case.fwd()
    for k in ("loss", "logp", "lse"):
        assert torch.equal(out[k], again[k]), k                              # run-to-run bitwise


def _oracle_grads(b, adv, old, grad_loss=None):
    head, _, _ = U.oracle_heads(b)
    return O.policy_loss_grads(b["H"], b["W"], b["target"], old, adv, b["resp_of_token"], head,
                               grad_loss=None if grad_loss is None else grad_loss.numpy())


@pytest.mark.parametrize("name", ["tiny", "mid", "mid_multi"])
@pytest.mark.parametrize("sigma", [0.05, 0.3])
def test_backward(name, sigma):
    b, lse, logp, adv, old = _case(name, sigma)
    M = b["spec"].n_heads
    gl = torch.tensor([1.0, 0.5, 2.0][:M]) if sigma > 0.1 else None
    case = U.PolicyCase(b, adv, old, grad_loss=gl)
    out = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    assert out["status"] == 0
    dH, dW = _oracle_grads(b, adv, old, gl)
    # whole-tensor relative Frobenius error AND a bound on every single row (token / vocabulary id)
    U.check_rows(out["dH"].numpy(), dH, "dH")
    for m in range(M):
        U.check_rows(out["dW"][m].numpy(), dW[m], "dW[%d]" % m)
    # rows that carry no gradient (clipped ratio or zero advantage) are exactly zero
    zero_rows = np.abs(dH).sum(1) == 0
    assert zero_rows.any() and (out["dH"].numpy()[zero_rows] == 0).all()
    # identities that hold at any size
    for m in range(M):
        col = out["dW"][m].double().sum(0).abs().max().item()
        assert col <= 1e-3 * out["dW"][m].double().abs().sum(0).max().item() + 1e-9


def test_backward_dtypes_and_accumulation():
    b, lse, logp, adv, old = _case("mid", 0.3)
    dH, dW = _oracle_grads(b, adv, old)
    lp, ls = torch.from_numpy(logp).float(), torch.from_numpy(lse).float()
    prm = A.Params(dH_dtype=A.F32, dW_dtype=A.BF16)
    out = U.PolicyCase(b, adv, old, prm=prm).bwd(lp, ls)
    assert U.rel_fro(out["dH"].numpy(), dH) <= 5e-3
    assert U.rel_fro(out["dW"][0].numpy(), dW[0]) <= 5e-3
    prm = A.Params(accumulate_dW=1)
    case = U.PolicyCase(b, adv, old, prm=prm)
    # accumulate twice into the same zero-initialised buffer through the raw call
    T, d, V = case.T, case.spec.d, case.spec.V
    dHb = torch.empty(T, d, dtype=torch.bfloat16, device=U.DEV)
    acc = [torch.zeros(V, d, dtype=torch.float32, device=U.DEV)]
    ws = A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, d, V, 1, True), U.DEV)
    st = A.new_status(U.DEV)
    for _ in range(2):
        A.atgrpo_policy_loss_bwd(case.H, case.W, case.target, None, None, case.resp_of_token, case.adv,
                                 case.old_logp, lp.to(U.DEV), ls.to(U.DEV), None, prm, dHb, acc, st, ws)
    torch.cuda.synchronize()
    assert U.rel_fro(acc[0].cpu().numpy(), 2 * dW[0]) <= 5e-3


def test_unused_head_and_tiny_T():
    # three heads, but every token belongs to roles that map to heads 0 and 2; T below one tile
    spec = WL.RolloutSpec("t", 1, 3, 1, 2, (5, 5, 5), (9, 9, 9), 64, 300, 3, 99, 0)
    b = WL.make_rollout(spec)
    b["head_of_role"] = torch.tensor([2, 0, 2], dtype=torch.int32)
    lse, logp = U.oracle_logprobs(b)
    adv = U.batch_advantages(b)
    old = U.keep_off_the_kinks(logp, WL.make_old_logp(torch.from_numpy(logp), 5, 0.3))
    case = U.PolicyCase(b, adv, old)
    out = case.fwd()
    head, offsets, perm = U.oracle_heads(b)
    assert np.array_equal(out["role_offsets"].numpy(), offsets) and np.array_equal(out["role_perm"].numpy(), perm)
    assert np.abs(out["logp"].numpy() - logp).max() <= 1e-3
    rloss, _, _ = O.policy_loss(logp, old, adv, b["resp_of_token"], head, 3)
    np.testing.assert_allclose(out["loss"].numpy(), rloss, rtol=1e-3, atol=1e-7)
    assert out["loss"][1] == 0
    g = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    dH, dW = _oracle_grads(b, adv, old)
    assert U.rel_fro(g["dH"].numpy(), dH) <= 5e-3
    assert (g["dW"][1] == 0).all()
    for m in (0, 2):
        assert U.rel_fro(g["dW"][m].numpy(), dW[m]) <= 5e-3


def test_bad_target_is_flagged_not_faulting():
    b, lse, logp, adv, old = _case("tiny", 0.05)
    b2 = dict(b)
    b2["target"] = b["target"].clone()
    b2["target"][17] = b["spec"].V + 5
    out = U.PolicyCase(b2, adv, old).fwd()
    assert out["status"] == A.ERR_BAD_INDEX
    keep = np.arange(b["T"]) != 17
    assert np.abs(out["logp"].numpy()[keep] - logp[keep]).max() <= 1e-3


def test_backward_is_bitwise_repeatable():
    # no floating-point atomics anywhere on the path: two runs give identical bits (doubles as a race check)
    b, lse, logp, adv, old = _case("mid_multi", 0.3)
    case = U.PolicyCase(b, adv, old)
    lp, ls = torch.from_numpy(logp).float(), torch.from_numpy(lse).float()
    a, c = case.bwd(lp, ls), case.bwd(lp, ls)
    assert torch.equal(a["dH"], c["dH"])
    for x, y in zip(a["dW"], c["dW"]):
        assert torch.equal(x, y)


def test_two_calls_on_two_streams_with_their_own_workspaces():
    # "calls may run concurrently on different streams if they use different workspaces and outputs":
    # two different batches, forward + backward each, enqueued on two streams without any ordering between
    # them, must give what each gives alone (one of them with kept logits)
    dev = U.DEV
    cases = []
    for name, keep in (("mid", True), ("mid_multi", False)):
        b, lse, logp, adv, old = _case(name, 0.3)
        c = U.PolicyCase(b, adv, old)
        if keep:
            c.lend_logits()
        alone_f = c.fwd(want_routing=False)
        alone_b = c.bwd(alone_f["logp"], alone_f["lse"])
        cases.append((b, c, alone_f, alone_b))
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = []
    torch.cuda.synchronize()
    for rep in range(3):
        outs.clear()
        for (b, c, f, _), st in zip(cases, streams):
            T, M, d, V = b["T"], c.M, c.spec.d, c.spec.V
            with torch.cuda.stream(st):
                o = dict(loss=torch.zeros(M, device=dev), logp=torch.zeros(T, device=dev), lse=torch.zeros(T, device=dev),
                         dH=torch.zeros(T, d, dtype=torch.bfloat16, device=dev),
                         dW=[torch.zeros(V, d, device=dev) for _ in range(M)], status=A.new_status(dev),
                         ws_f=A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, d, V, M, False), dev),
                         ws_b=A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, d, V, M, True), dev))
                outs.append(o)
        for (b, c, f, _), st, o in zip(cases, streams, outs):
            with torch.cuda.stream(st):
                A.atgrpo_policy_loss_fwd(c.H, c.W, c.target, c.role_of_token, c.head_of_role, c.resp_of_token, c.adv,
                                         c.old_logp, c.prm, o["loss"], o["logp"], o["lse"], device_status=o["status"],
                                         workspace=o["ws_f"])
        for (b, c, f, _), st, o in zip(cases, streams, outs):
            with torch.cuda.stream(st):
                A.atgrpo_policy_loss_bwd(c.H, c.W, c.target, c.role_of_token, c.head_of_role, c.resp_of_token, c.adv,
                                         c.old_logp, o["logp"], o["lse"], None, c.prm, o["dH"], o["dW"],
                                         device_status=o["status"], workspace=o["ws_b"])
        torch.cuda.synchronize()
        for (b, c, f, g), o in zip(cases, outs):
            assert int(o["status"].item()) == 0
            assert torch.equal(o["logp"].cpu(), f["logp"]) and torch.equal(o["loss"].cpu(), f["loss"])
            assert torch.equal(o["dH"].float().cpu(), g["dH"])
            for m in range(c.M):
                assert torch.equal(o["dW"][m].cpu(), g["dW"][m])
