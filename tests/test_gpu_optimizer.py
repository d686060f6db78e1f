"""CUDA gradient-norm and AdamW update vs. the fp64 oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

from oracle import atgrpo_oracle as O
from paper_2510_11062_b200 import atgrpo as A
from tests import _util as U

pytestmark = pytest.mark.gpu


def _sumsq(grad):
    dev = U.DEV
    out = torch.zeros(1, dtype=torch.float64, device=dev)
    ws = A.workspace(A.atgrpo_grad_sumsq_workspace_bytes(), dev)
    A.atgrpo_grad_sumsq(grad.to(dev), out, ws)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("n", [1, 7, 8, 1000003])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_grad_sumsq(n, dtype):
    g = torch.Generator().manual_seed(n)
    grad = (torch.randn(n, generator=g) * 3).to(dtype)
    got = _sumsq(grad).item()
    assert got == pytest.approx(O.grad_sumsq([grad]), rel=1e-6)
    assert got == _sumsq(grad).item()                         # fixed order: bitwise repeatable


@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_adamw_steps_vs_oracle(gdtype):
    dev = U.DEV
    n = 300007                                               # ragged tail for the 8-wide main loop
    g = torch.Generator().manual_seed(17)
    theta0 = torch.randn(n, generator=g) * 0.05
    master, m, v = theta0.clone().to(dev), torch.zeros(n, device=dev), torch.zeros(n, device=dev)
    w = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    th, mo, vo = theta0.double().numpy(), np.zeros(n), np.zeros(n)
    ws = A.workspace(A.atgrpo_grad_sumsq_workspace_bytes(), dev)
    sumsq = torch.zeros(1, dtype=torch.float64, device=dev)
    for step in range(1, 5):
        grad = (torch.randn(n, generator=g) * (0.05 if step != 2 else 1e-4)).to(gdtype)
        prm = A.AdamWParams(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.01, max_grad_norm=1.0, step=step)
        gd = grad.to(dev)
        A.atgrpo_grad_sumsq(gd, sumsq, ws)
        A.atgrpo_adamw_step(gd, master, m, v, w, sumsq, prm)
        scale = O.clip_scale(O.grad_sumsq([grad]), 1.0)
        th, mo, vo = O.adamw_step(th, mo, vo, grad, step, lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8,
                                  weight_decay=0.01, scale=scale)
        if step == 1:
            assert scale < 1.0                                 # clipping active on the big-gradient steps
    torch.cuda.synchronize()
    assert U.rel_fro(master.cpu().numpy(), th) <= 1e-5
    np.testing.assert_allclose(m.cpu().numpy(), mo, rtol=1e-4, atol=1e-9)
    np.testing.assert_allclose(v.cpu().numpy(), vo, rtol=1e-4, atol=1e-12)
    assert torch.equal(w.cpu(), master.cpu().to(torch.bfloat16))   # the bf16 head is the rounded master


def test_adamw_without_clipping_and_without_bf16_copy():
    dev = U.DEV
    n = 4096
    g = torch.Generator().manual_seed(3)
    theta0, grad = torch.randn(n, generator=g), torch.randn(n, generator=g) * 50
    master, m, v = theta0.clone().to(dev), torch.zeros(n, device=dev), torch.zeros(n, device=dev)
    prm = A.AdamWParams(lr=1e-2, max_grad_norm=0.0, step=1)
    A.atgrpo_adamw_step(grad.to(dev), master, m, v, None, None, prm)
    torch.cuda.synchronize()
    th, _, _ = O.adamw_step(theta0, np.zeros(n), np.zeros(n), grad, 1, lr=1e-2)
    assert U.rel_fro(master.cpu().numpy(), th) <= 1e-6
