"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The fp64 oracle cannot afford the full [T, V] softmax at these sizes, so the cases are built such
that everything the library outputs is still checkable against it:
  * lse / logp on a random sample of tokens (each needs only its own logit row);
  * advantages are made SPARSE (non-zero for a few responses spread over the batch), so loss, the
    dH rows of those responses and the COMPLETE dW of every head depend only on tokens the oracle
    can afford; all other dH rows must be exactly zero.  The backward routes only tokens with a
    non-zero gradient factor, so these cases run few row tiles but EVERY vocabulary tile and chunk:
    they are the complete-dW check (every one of the V rows of every head is compared), also with
    accumulation over two micro-batches.  The dense-advantage run of every row tile is compared
    with the oracle on sampled rows in test_gpu_full_size_dense.py;
  * identities that hold at any size on a dense-advantage run (column sums of dW, <dH,H> = <dW,W>).
The memory-bound stress input is compared in full."""
import numpy as np
import pytest
import torch

from oracle import atgrpo_oracle as O
from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu


def _sparse_case(name, n_active_resp=6, n_sample=160, shift=0, batch=None):
    b = batch if batch is not None else WL.make_rollout(WL.SPECS[name])
    spec, T, R, M = b["spec"], b["T"], b["R"], b["spec"].n_heads
    g = torch.Generator().manual_seed(spec.seed + 7)
    head, offsets, perm = U.oracle_heads(b)
    # a few responses spread over the batch (and over the roles) carry a non-zero advantage
    active_resp = torch.linspace(1, R - 2, n_active_resp).long() + torch.arange(n_active_resp) % spec.n_role
    active_resp = torch.unique((active_resp + shift).clamp(max=R - 1))
    adv = torch.zeros(R, dtype=torch.float64)
    adv[active_resp] = torch.tensor([1.0, -0.7, 0.45, -1.3, 0.8, -0.25, 0.6, -0.9])[: active_resp.numel()].double()
    resp = b["resp_of_token"].long()
    act = torch.nonzero(adv[resp] != 0).squeeze(1).numpy()
    sample = np.unique(np.concatenate([act, torch.randint(0, T, (n_sample,), generator=g).numpy(),
                                       [0, T - 1]]))
    lse_s, logp_s = np.zeros(sample.size), np.zeros(sample.size)
    for m in range(M):
        sel = head[sample] == m
        if sel.any():
            lse_s[sel], logp_s[sel], _ = O.token_logprobs(b["H"][sample[sel]], b["W"][m], b["target"][sample[sel]])
    pos = {int(t): i for i, t in enumerate(sample)}
    act_pos = np.array([pos[int(t)] for t in act])
    old = torch.full((T,), -9.0)
    noise = torch.randn(act.size, generator=g) * 0.3
    old_act = U.keep_off_the_kinks(logp_s[act_pos], torch.from_numpy(logp_s[act_pos]).float() + noise)
    old[torch.from_numpy(act)] = old_act
    return dict(b=b, head=head, offsets=offsets, perm=perm, adv=adv, act=act, sample=sample, lse_s=lse_s,
                logp_s=logp_s, act_pos=act_pos, old=old)


@pytest.mark.parametrize("name", ["qwen3_1p7b", "multi3", "qwen3_8b", "long_resp"])
def test_full_size_sparse_advantages(name):
    c = _sparse_case(name, n_active_resp=2) if name == "long_resp" else _sparse_case(name)
    b, head, act, M = c["b"], c["head"], c["act"], c["b"]["spec"].n_heads
    case = U.PolicyCase(b, c["adv"], c["old"])
    case.lend_logits()                                    # the timed configuration: logits kept by the forward
    out = case.fwd()
    assert out["status"] == 0
    assert np.array_equal(out["role_offsets"].numpy(), c["offsets"])
    assert np.array_equal(out["role_perm"].numpy(), c["perm"])
    assert np.abs(out["lse"].numpy()[c["sample"]] - c["lse_s"]).max() <= 1e-3
    assert np.abs(out["logp"].numpy()[c["sample"]] - c["logp_s"]).max() <= 1e-3
    # loss: only the active tokens contribute; the denominator is every token of the head
    T_m = np.bincount(head, minlength=M).astype(np.float64)
    n_act = np.bincount(head[act], minlength=M).astype(np.float64)
    resp_act = b["resp_of_token"][torch.from_numpy(act)]
    sub_loss, _, _ = O.policy_loss(c["logp_s"][c["act_pos"]], c["old"][torch.from_numpy(act)], c["adv"], resp_act,
                                   head[act], M)
    want_loss = sub_loss * n_act / np.maximum(T_m, 1)
    np.testing.assert_allclose(out["loss"].numpy(), want_loss, rtol=1e-3, atol=1e-9)
    # backward, fed with the oracle's log-probs where they matter
    logp_in = torch.zeros(b["T"])
    lse_in = torch.from_numpy(np.full(b["T"], 12.0, dtype=np.float32))
    logp_in[torch.from_numpy(c["sample"])] = torch.from_numpy(c["logp_s"]).float()
    lse_in[torch.from_numpy(c["sample"])] = torch.from_numpy(c["lse_s"]).float()
    g = case.bwd_both_ways(logp_in, lse_in)               # from the kept logits, and recomputed: same bits
    assert g["status"] == 0
    ta = torch.from_numpy(act)
    dH_act, dW = O.policy_loss_grads(b["H"][ta], b["W"], b["target"][ta], c["old"][ta], c["adv"], resp_act,
                                     head[act], grad_loss=n_act / np.maximum(T_m, 1))
    dH = g["dH"].numpy()
    assert U.rel_fro(dH[act], dH_act) <= 5e-3
    rest = np.ones(b["T"], bool)
    rest[act] = False
    assert (dH[rest] == 0).all()
    for m in range(M):
        assert U.rel_fro(g["dW"][m].numpy(), dW[m]) <= 5e-3, m
    if name in ("qwen3_8b", "long_resp"):
        # the same from logits kept as 16-bit codes (d = 4096 / the longest batch): the oracle's tolerances again
        case.lend_logits(A.LOGITS_Q16)
        assert case.fwd()["status"] == 0
        g16 = case.bwd(logp_in, lse_in)
        assert g16["status"] == 0
        assert U.rel_fro(g16["dH"].numpy()[act], dH_act) <= 5e-3 and (g16["dH"].numpy()[rest] == 0).all()
        for m in range(M):
            assert U.rel_fro(g16["dW"][m].numpy(), dW[m]) <= 5e-3, m


@pytest.mark.parametrize("dw_dtype", [A.F32, A.BF16])
def test_full_size_accumulation_over_two_micro_batches(dw_dtype):
    # gradient accumulation (App. "Training Details": a global batch is several mini-batches): two
    # micro-batches with different active responses are accumulated into ONE dW at the full
    # vocabulary (10 chunks), and the sum is compared row by row with the oracle's summed gradient
    name = "qwen3_1p7b"
    b = WL.make_rollout(WL.SPECS[name])
    cases = [_sparse_case(name, n_active_resp=4, n_sample=8, shift=0, batch=b),
             _sparse_case(name, n_active_resp=4, n_sample=8, shift=5, batch=b)]
    T, d, V = b["T"], b["spec"].d, b["spec"].V
    dev = U.DEV
    prm = A.Params(accumulate_dW=1, dW_dtype=dw_dtype)
    acc = [torch.zeros(V, d, dtype=torch.float32 if dw_dtype == A.F32 else torch.bfloat16, device=dev)]
    ws = A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, d, V, 1, True), dev)
    st = A.new_status(dev)
    dH = torch.empty(T, d, dtype=torch.bfloat16, device=dev)
    want = np.zeros((V, d))
    for c in cases:
        case = U.PolicyCase(c["b"], c["adv"], c["old"], prm=prm)
        logp_in = torch.zeros(T)
        lse_in = torch.full((T,), 12.0)
        logp_in[torch.from_numpy(c["sample"])] = torch.from_numpy(c["logp_s"]).float()
        lse_in[torch.from_numpy(c["sample"])] = torch.from_numpy(c["lse_s"]).float()
        A.atgrpo_policy_loss_bwd(case.H, case.W, case.target, None, None, case.resp_of_token, case.adv,
                                 case.old_logp, logp_in.to(dev), lse_in.to(dev), None, prm, dH, acc, st, ws)
        ta = torch.from_numpy(c["act"])
        n_act = float(c["act"].size)
        _, dW = O.policy_loss_grads(b["H"][ta], b["W"], b["target"][ta], c["old"][ta], c["adv"],
                                    b["resp_of_token"][ta], np.zeros(c["act"].size, dtype=np.int64),
                                    grad_loss=np.array([n_act / T]))
        want += dW[0]
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert not np.array_equal(cases[0]["act"], cases[1]["act"])
    U.check_rows(acc[0].float().cpu().numpy(), want, "accumulated dW", row_rel=1.5e-2 if dw_dtype == A.BF16 else 1e-2)


def test_full_size_dense_identities():
    # dense advantages at the benchmark size: identities that need no oracle
    b = WL.make_rollout(WL.SPECS["qwen3_1p7b"])
    adv = U.batch_advantages(b)
    case = U.PolicyCase(b, adv, torch.zeros(b["T"]))
    out = case.fwd()
    old = WL.make_old_logp(out["logp"], 3, 0.3)           # perf-style input: only identities are checked
    case = U.PolicyCase(b, adv, old)
    out2 = case.fwd()
    assert torch.equal(out["logp"], out2["logp"]) and torch.equal(out["lse"], out2["lse"])
    g = case.bwd(out2["logp"], out2["lse"])
    assert g["status"] == 0
    dW, dH = g["dW"][0].double(), g["dH"].double()
    assert dW.sum(0).abs().max().item() <= 2e-3 * dW.abs().sum(0).max().item()      # sum_v dZ_jv = 0
    lhs = (dH * b["H"].double()).sum().item()
    rhs = (dW * b["W"][0].double()).sum().item()
    scale = (dH.norm() * b["H"].double().norm()).item()
    assert abs(lhs - rhs) <= 5e-3 * scale
    p = out2["logp"].double().exp()
    assert ((p > 0) & (p <= 1.0 + 1e-6)).all()


def test_stress_full_size():
    s = WL.make_stress()
    dims = (s["n_env"], s["n_role"], s["n_turn"])
    ref = U.oracle_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], *dims)
    for bucketing in (False, True):
        gpu = U.gpu_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], *dims,
                                     bucketing=bucketing)
        U.check_group_advantages(gpu, ref)
    assert (ref["adv"] == 0).sum() > 0.01 * s["G"]
    adv = torch.from_numpy(ref["adv"]).float()
    dev = U.DEV
    loss = torch.zeros(1, device=dev)
    cc = torch.zeros(2, dtype=torch.int64, device=dev)
    st = A.new_status(dev)
    old = U.keep_off_the_kinks(s["logp"].numpy(), s["old_logp"])
    A.atgrpo_clipped_loss(s["logp"].to(dev), old.to(dev), s["resp_of_token"].to(dev), adv.to(dev), A.Params(), loss,
                          None, cc, st, A.workspace(A.atgrpo_clipped_loss_workspace_bytes(s["T"]), dev))
    torch.cuda.synchronize()
    rl, _, rcc = O.policy_loss(s["logp"], old, adv, s["resp_of_token"], np.zeros(s["T"], int), 1)
    assert int(st.item()) == 0
    assert abs(loss.item() - rl[0]) <= 1e-3 * abs(rl[0])
    assert np.abs(cc.cpu().numpy() - rcc[0]).max() <= 2
