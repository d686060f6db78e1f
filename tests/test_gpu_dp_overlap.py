"""Backward with a notification per vocabulary chunk (atgrpo_policy_loss_bwd_notify) and the
overlapped all-reduce built on it: same gradients as the plain backward call, bit for bit, every
event recorded, and the chunk-wise all-reduce (one rank, NCCL) leaves the sum in dW."""
import os

import pytest
import torch
import torch.distributed as dist

from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import data_parallel as DP
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu

# three roles with their own heads and a vocabulary wide enough for several chunks at a small d
SPEC = WL.RolloutSpec("dp_overlap", 6, 3, 2, 4, (24, 8, 8), (40, 24, 24), 64, 151936, 3, 1251)


def _case():
    b = WL.make_rollout(SPEC)
    adv = torch.where(torch.arange(b["R"]) % 5 == 0, 0.0, 1.0) * (torch.arange(b["R"]) % 7 - 3.0)
    case = U.PolicyCase(b, adv, torch.zeros(b["T"]))
    f = case.fwd(want_routing=False)
    assert f["status"] == 0
    case.old_logp = (f["logp"] + 0.3 * torch.sin(torch.arange(b["T"]).float())).to(U.DEV)
    return b, case, f


def _bwd_kwargs(case, f, dH, dW, status, ws):
    return dict(H=case.H, W=case.W, target=case.target, role_of_token=case.role_of_token,
                head_of_role=case.head_of_role, resp_of_token=case.resp_of_token, adv=case.adv,
                old_logp=case.old_logp, logp=f["logp"].to(U.DEV), lse=f["lse"].to(U.DEV), grad_loss=None,
                params=case.prm, dH=dH, dW=dW, device_status=status, workspace=ws)


def test_notify_matches_plain_backward_and_overlapped_allreduce():
    b, case, f = _case()
    T, d, V, M = b["T"], SPEC.d, SPEC.V, SPEC.n_heads
    n_chunks, rows = A.atgrpo_policy_loss_bwd_chunks(T, d, V, M)
    assert n_chunks >= 2 and rows % 256 == 0 and (n_chunks - 1) * rows < V <= n_chunks * rows
    ranges = DP.chunk_row_ranges(V, n_chunks, rows)
    assert ranges[0][0] == 0 and ranges[-1][1] == V and all(a[1] == b_[0] for a, b_ in zip(ranges, ranges[1:]))

    ref = case.bwd(f["logp"], f["lse"])
    assert ref["status"] == 0

    ws = A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, d, V, M, True), U.DEV)
    status = A.new_status(U.DEV)
    mk = lambda: (torch.full((T, d), 7.0, dtype=torch.bfloat16, device=U.DEV),
                  [torch.full((V, d), 7.0, dtype=torch.float32, device=U.DEV) for _ in range(M)])

    # (1) events only
    dH, dW = mk()
    events = [torch.cuda.Event() for _ in range(n_chunks)]
    A.atgrpo_policy_loss_bwd(**_bwd_kwargs(case, f, dH, dW, status, ws), chunk_events=events)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and all(ev.query() for ev in events)
    assert torch.equal(dH.float().cpu(), ref["dH"])
    for m in range(M):
        assert torch.equal(dW[m].cpu(), ref["dW"][m])

    # a wrong number of events is refused on the host
    with pytest.raises(A.AtgrpoError):
        A.atgrpo_policy_loss_bwd(**_bwd_kwargs(case, f, dH, dW, status, ws), chunk_events=events[:-1])

    # (2) chunk-wise all-reduce on a second stream, one rank: the sum over ranks is the local gradient
    created = False
    if not dist.is_initialized():
        port = 29600 + os.getpid() % 300
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                                device_id=torch.device(U.DEV))
        created = True
    try:
        dH2, dW2 = mk()
        comm = torch.cuda.Stream()
        DP.backward_overlapped(A, _bwd_kwargs(case, f, dH2, dW2, status, ws), comm)
        # the main stream waits for the communication stream: work enqueued now sees the summed rows
        total = sum(w.double().sum() for w in dW2)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for m in range(M):
            assert torch.equal(dW2[m].cpu(), ref["dW"][m])
        assert torch.equal(dH2.float().cpu(), ref["dH"])
        assert float(total) == float(sum(w.double().sum() for w in ref["dW"]))
    finally:
        if created:
            dist.destroy_process_group()


def test_notify_with_no_tokens_records_every_event():
    d, V, M = 64, 1000, 1
    n_chunks, _ = A.atgrpo_policy_loss_bwd_chunks(0, d, V, M)
    z = lambda dt: torch.zeros(0, dtype=dt, device=U.DEV)
    W = [torch.zeros(V, d, dtype=torch.bfloat16, device=U.DEV)]
    dW = [torch.full((V, d), 3.0, dtype=torch.float32, device=U.DEV)]
    events = [torch.cuda.Event() for _ in range(n_chunks)]
    ws = A.workspace(A.atgrpo_policy_loss_workspace_bytes(0, d, V, M, True), U.DEV)
    A.atgrpo_policy_loss_bwd(torch.zeros(0, d, dtype=torch.bfloat16, device=U.DEV), W, z(torch.int32), None, None,
                             z(torch.int32), z(torch.float32), z(torch.float32), z(torch.float32),
                             z(torch.float32), None, A.Params(), torch.zeros(0, d, dtype=torch.bfloat16, device=U.DEV),
                             dW, device_status=A.new_status(U.DEV), workspace=ws, chunk_events=events)
    torch.cuda.synchronize()
    assert all(ev.query() for ev in events) and (dW[0] == 0).all()


def test_multi_chunk_multi_head_configuration_matches_the_oracle():
    # the configuration of this file (three heads, a vocabulary walked in several chunks, d = 64) with
    # old_logp built from the ORACLE's log-probs: forward, loss and the complete dH / dW of every head
    import numpy as np
    from oracle import atgrpo_oracle as O
    b = WL.make_rollout(SPEC)
    T, d, V, M = b["T"], SPEC.d, SPEC.V, SPEC.n_heads
    n_chunks, _ = A.atgrpo_policy_loss_bwd_chunks(T, d, V, M)
    assert n_chunks >= 2
    lse, logp = U.oracle_logprobs(b, chunk=1024)
    adv = U.batch_advantages(b)
    old = U.keep_off_the_kinks(logp, WL.make_old_logp(torch.from_numpy(logp), 17, 0.3))
    head, offsets, perm = U.oracle_heads(b)
    gl = torch.tensor([1.0, 0.5, 2.0])
    case = U.PolicyCase(b, adv, old, grad_loss=gl)
    out = case.fwd()
    assert out["status"] == 0
    assert np.abs(out["lse"].numpy() - lse).max() <= 1e-3 and np.abs(out["logp"].numpy() - logp).max() <= 1e-3
    rl, _, _ = O.policy_loss(logp, old, adv, b["resp_of_token"], head, M)
    np.testing.assert_allclose(out["loss"].numpy(), rl, rtol=1e-3)
    g = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    assert g["status"] == 0
    dH, dW = O.policy_loss_grads(b["H"], b["W"], b["target"], old, adv, b["resp_of_token"], head, grad_loss=gl.numpy())
    U.check_rows(g["dH"].numpy(), dH, "dH")
    for m in range(M):
        U.check_rows(g["dW"][m].numpy(), dW[m], "dW[%d]" % m)
