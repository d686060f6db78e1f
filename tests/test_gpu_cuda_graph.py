"""One whole step -- advantages, forward, backward (logits kept) -- captured into a CUDA graph: the
library allocates nothing, never synchronises, sizes every launch from (T, d, V, M) on the host and
takes everything that depends on the data (routing, which rows carry a gradient) on the device, so a
captured step can be replayed on new inputs written into the same buffers."""
import pytest
import torch

from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu


def test_a_captured_step_replays_bit_for_bit_also_on_new_inputs():
    dev = U.DEV
    b = WL.make_rollout(WL.SPECS["mid_multi"])
    s = b["spec"]
    T, R, d, V, M = b["T"], b["R"], s.d, s.V, s.n_heads
    G = s.n_env * s.n_role * s.n_turn
    g = {k: b[k].to(dev) for k in ("rewards", "env_id", "role_id", "turn_id", "H", "target", "resp_of_token",
                                   "role_of_token")}
    W = [w.to(dev) for w in b["W"]]
    hor = b["head_of_role"].to(dev)
    adv, loss = torch.zeros(R, device=dev), torch.zeros(M, device=dev)
    logp, lse, old = torch.zeros(T, device=dev), torch.zeros(T, device=dev), torch.zeros(T, device=dev)
    dH = torch.zeros(T, d, dtype=torch.bfloat16, device=dev)
    dW = [torch.zeros(V, d, device=dev) for _ in range(M)]
    st = A.new_status(dev)
    ws_a = A.workspace(A.atgrpo_group_advantages_workspace_bytes(R, G), dev)
    ws_f = A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, d, V, M, False), dev)
    ws_b = A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, d, V, M, True), dev)
    prm = A.Params(logits=torch.empty(A.atgrpo_policy_loss_logits_bytes(T, V) // 4, device=dev))

    def step():
        A.atgrpo_group_advantages(g["rewards"], g["env_id"], g["role_id"], g["turn_id"], s.n_env, s.n_role, s.n_turn,
                                  prm, adv, device_status=st, workspace=ws_a)
        A.atgrpo_policy_loss_fwd(g["H"], W, g["target"], g["role_of_token"], hor, g["resp_of_token"], adv, old, prm,
                                 loss, logp, lse, device_status=st, workspace=ws_f)
        A.atgrpo_policy_loss_bwd(g["H"], W, g["target"], g["role_of_token"], hor, g["resp_of_token"], adv, old, logp,
                                 lse, None, prm, dH, dW, device_status=st, workspace=ws_b)

    def snapshot():
        torch.cuda.synchronize()
        return dH.clone(), [w.clone() for w in dW], loss.clone(), adv.clone()

    def same(x, y):
        return torch.equal(x[0], y[0]) and all(torch.equal(p, q) for p, q in zip(x[1], y[1])) and \
            torch.equal(x[2], y[2]) and torch.equal(x[3], y[3])

    step()                                       # first call: the library looks up the tensor-map encoder once
    torch.cuda.synchronize()
    old.copy_(logp + 0.3 * torch.sin(torch.arange(T, device=dev).float()))
    step()
    eager = snapshot()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for t in (dH, loss, adv, *dW):
        t.fill_(7.0)
    graph.replay()
    assert same(snapshot(), eager) and int(st.item()) == 0 and float(dW[0].abs().max()) > 0
    # new inputs in the same buffers: other hidden states, other rewards (so other tokens carry a gradient)
    g["H"].copy_((b["H"].float() * 0.5).to(torch.bfloat16))
    g["rewards"].copy_(torch.roll(b["rewards"], 5))
    graph.replay()
    replayed = snapshot()
    step()
    assert same(snapshot(), replayed) and not same(replayed, eager) and int(st.item()) == 0
