"""Helpers shared by the GPU parity tests: run the CUDA library and the fp64 oracle on the same
seeded inputs.  The oracle never receives anything the CUDA path produced."""
from __future__ import annotations

import numpy as np
import torch

from oracle import atgrpo_oracle as O
from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL

DEV = "cuda:0"


def rel_fro(x, ref):
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(x - ref) / den) if den > 0 else float(np.linalg.norm(x))


def to_dev(t):
    return None if t is None else t.to(DEV)


def gpu_group_advantages(rewards, env_id, role_id, turn_id, n_env, n_role, n_turn, prm=None,
                         want_all=True, bucketing=True):
    """bucketing=False leaves group_offsets / group_perm out, which selects the library's sort-free
    pipeline; with them it runs the counting-sort pipeline."""
    prm = prm or A.Params()
    R, G = rewards.numel(), n_env * n_role * n_turn
    i32, f32 = torch.int32, torch.float32
    out = dict(adv=torch.full((R,), 7.0, dtype=f32, device=DEV))
    if want_all:
        out.update(group_of_cand=torch.full((R,), -5, dtype=i32, device=DEV),
                   group_mean=torch.full((G,), 7.0, dtype=f32, device=DEV),
                   group_std=torch.full((G,), 7.0, dtype=f32, device=DEV))
        if bucketing:
            out.update(group_offsets=torch.full((G + 1,), -5, dtype=i32, device=DEV),
                       group_perm=torch.full((R,), -5, dtype=i32, device=DEV))
    status = A.new_status(DEV)
    ws = A.workspace(A.atgrpo_group_advantages_workspace_bytes(R, G), DEV)
    A.atgrpo_group_advantages(to_dev(rewards), to_dev(env_id), to_dev(role_id), to_dev(turn_id),
                              n_env, n_role, n_turn, prm, device_status=status, workspace=ws, **out)
    torch.cuda.synchronize()
    out = {k: v.cpu() for k, v in out.items()}
    out["status"] = int(status.item())
    return out


def oracle_group_advantages(rewards, env_id, role_id, turn_id, n_env, n_role, n_turn, eps=1e-6, ddof=0):
    G = n_env * n_role * n_turn
    key = O.group_key(env_id, role_id, turn_id, n_env, n_role, n_turn)
    offsets, perm = O.bucket_by_key(key, G)
    adv, mean, std = O.group_advantages(rewards, key, G, eps, ddof)
    return dict(adv=adv, group_of_cand=key, group_offsets=offsets, group_perm=perm,
                group_mean=mean, group_std=std)


def check_group_advantages(gpu, ref):
    assert gpu["status"] == 0
    for k in ("group_of_cand", "group_offsets", "group_perm"):
        if k in gpu:
            assert np.array_equal(gpu[k].numpy().astype(np.int64), ref[k]), k      # bit-exact
    a, r = gpu["adv"].numpy().astype(np.float64), ref["adv"]
    assert (np.abs(a - r) <= 1e-5 * np.maximum(1.0, np.abs(r))).all()
    assert (a[r == 0.0] == 0.0).all()                  # all-equal and K=1 groups: exact zeros
    if "group_mean" in gpu:
        np.testing.assert_allclose(gpu["group_mean"].numpy(), ref["group_mean"], rtol=1e-6, atol=1e-7)
        np.testing.assert_allclose(gpu["group_std"].numpy(), ref["group_std"], rtol=1e-6, atol=1e-7)


class PolicyCase:
    """One rollout batch on the GPU plus the oracle's view of it."""

    def __init__(self, batch, adv, old_logp, prm=None, grad_loss=None):
        self.b = batch
        self.spec = batch["spec"]
        self.M = self.spec.n_heads
        self.prm = prm or A.Params()
        self.T = batch["T"]
        self.H = to_dev(batch["H"])
        self.W = [to_dev(w) for w in batch["W"]]
        self.target = to_dev(batch["target"])
        self.multi = self.M > 1
        self.role_of_token = to_dev(batch["role_of_token"]) if self.multi else None
        self.head_of_role = to_dev(batch["head_of_role"]) if self.multi else None
        self.resp_of_token = to_dev(batch["resp_of_token"])
        self.adv = to_dev(adv.to(torch.float32))
        self.old_logp = to_dev(old_logp.to(torch.float32))
        self.grad_loss = None if grad_loss is None else to_dev(grad_loss.to(torch.float32))

    def lend_logits(self, fmt=A.LOGITS_F32):
        """Lends the library a logits buffer (params.logits) full of NaN (fp32 format) or of 0xFF bytes
        (16-bit codes: every code saturated, every block maximum a NaN): the next forward stores the
        logits there and the backward calls after it read them instead of recomputing.  Whatever the
        library leaves unwritten must never reach a result."""
        import dataclasses
        n = A.atgrpo_policy_loss_logits_bytes(self.T, self.spec.V, fmt)
        if fmt == A.LOGITS_F32:
            buf = torch.full((n // 4,), float("nan"), dtype=torch.float32, device=DEV)
        else:
            buf = torch.full((n,), 255, dtype=torch.uint8, device=DEV)
        self.prm = dataclasses.replace(self.prm, logits=buf, logits_format=fmt)
        return buf

    def bwd_both_ways(self, logp, lse):
        """Backward from the kept logits (lend_logits() and fwd() came first) and again with the
        contraction recomputed: the two must agree bit for bit.  Returns the first."""
        import dataclasses
        assert self.prm.logits is not None
        kept = self.bwd(logp, lse)
        lent = self.prm
        self.prm = dataclasses.replace(lent, logits=None)
        again = self.bwd(logp, lse)
        self.prm = lent
        assert again["status"] == kept["status"]
        assert torch.equal(kept["dH"], again["dH"]), "dH: kept logits vs recomputed"
        for m in range(self.M):
            assert torch.equal(kept["dW"][m], again["dW"][m]), ("dW: kept logits vs recomputed", m)
        return kept

    def fwd(self, want_routing=True):
        f32, i32 = torch.float32, torch.int32
        T, M = self.T, self.M
        out = dict(loss=torch.full((M,), 7.0, dtype=f32, device=DEV),
                   logp=torch.full((T,), 7.0, dtype=f32, device=DEV),
                   lse=torch.full((T,), 7.0, dtype=f32, device=DEV),
                   clip_counts=torch.full((M, 2), -1, dtype=torch.int64, device=DEV))
        if want_routing:
            out.update(role_offsets=torch.full((M + 1,), -5, dtype=i32, device=DEV),
                       role_perm=torch.full((T,), -5, dtype=i32, device=DEV))
        status = A.new_status(DEV)
        ws = A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, self.spec.d, self.spec.V, M, False), DEV)
        A.atgrpo_policy_loss_fwd(self.H, self.W, self.target, self.role_of_token, self.head_of_role,
                                 self.resp_of_token, self.adv, self.old_logp, self.prm,
                                 device_status=status, workspace=ws, **out)
        torch.cuda.synchronize()
        res = {k: v.cpu() for k, v in out.items()}
        res["status"] = int(status.item())
        return res

    def bwd(self, logp, lse):
        f32, bf = torch.float32, torch.bfloat16
        T, M, d, V = self.T, self.M, self.spec.d, self.spec.V
        dH = torch.full((T, d), 7.0, dtype=bf if self.prm.dH_dtype == A.BF16 else f32, device=DEV)
        dwt = bf if self.prm.dW_dtype == A.BF16 else f32
        dW = [torch.full((V, d), 7.0 if not self.prm.accumulate_dW else 0.0, dtype=dwt, device=DEV)
              for _ in range(M)]
        status = A.new_status(DEV)
        ws = A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, d, V, M, True), DEV)
        A.atgrpo_policy_loss_bwd(self.H, self.W, self.target, self.role_of_token, self.head_of_role,
                                 self.resp_of_token, self.adv, self.old_logp, to_dev(logp), to_dev(lse),
                                 self.grad_loss, self.prm, dH, dW, device_status=status, workspace=ws)
        torch.cuda.synchronize()
        return dict(dH=dH.float().cpu(), dW=[w.float().cpu() for w in dW], status=int(status.item()))


def oracle_heads(batch):
    spec = batch["spec"]
    if spec.n_heads == 1:
        T = batch["T"]
        return np.zeros(T, dtype=np.int64), np.array([0, T]), np.arange(T)
    return O.route_tokens(batch["role_of_token"], batch["head_of_role"], spec.n_heads)


def oracle_logprobs(batch, chunk=2048):
    """lse, logp for every token (rows are independent, so the oracle is called on row slices)."""
    head, _, _ = oracle_heads(batch)
    T = batch["T"]
    lse, logp = np.zeros(T), np.zeros(T)
    for m in range(batch["spec"].n_heads):
        sel = np.nonzero(head == m)[0]
        for s in range(0, sel.size, chunk):
            idx = sel[s:s + chunk]
            l, p, _ = O.token_logprobs(batch["H"][idx], batch["W"][m], batch["target"][idx])
            lse[idx], logp[idx] = l, p
    return lse, logp


def batch_advantages(batch):
    spec = batch["spec"]
    ref = oracle_group_advantages(batch["rewards"], batch["env_id"], batch["role_id"], batch["turn_id"],
                                  spec.n_env, spec.n_role, spec.n_turn)
    return torch.from_numpy(ref["adv"])


def keep_off_the_kinks(logp, old_logp, eps_lo=0.2, eps_hi=0.2, margin=2e-3):
    """Moves old_logp of the few tokens whose ratio sits within `margin` of a clip boundary so that
    fp32 and fp64 take the same clip decision (the gradient is discontinuous there)."""
    rho = np.exp(np.asarray(logp, np.float64) - old_logp.double().numpy())
    near = (np.abs(rho - (1 - eps_lo)) < margin) | (np.abs(rho - (1 + eps_hi)) < margin)
    out = old_logp.clone()
    out[torch.from_numpy(near)] = torch.from_numpy(np.asarray(logp, np.float32))[torch.from_numpy(near)]
    return out


def check_rows(x, ref, what, fro=5e-3, row_rel=1e-2, row_abs=1e-3):
    """Gradient rows against the oracle's: the relative Frobenius error of the whole block (the
    stated tolerance) AND a bound per row, |x_r - ref_r| <= row_rel*|ref_r| + row_abs*rms_r|ref_r|,
    so that a single wrong row cannot hide inside the norm of a large block."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert x.shape == ref.shape, what
    assert rel_fro(x, ref) <= fro, (what, rel_fro(x, ref))
    norms = np.linalg.norm(ref, axis=1)
    err = np.linalg.norm(x - ref, axis=1)
    rms = float(np.sqrt((norms ** 2).mean())) if norms.size else 0.0
    bound = row_rel * norms + row_abs * rms
    worst = int(np.argmax(err - bound)) if err.size else 0
    assert (err <= bound).all(), (what, "row", worst, float(err[worst]), float(bound[worst]))
    zero = norms == 0.0
    assert (x[zero] == 0.0).all(), (what, "rows that carry no gradient must be exactly zero")


def oracle_logprobs_cached(batch, pytest_cache):
    """oracle_logprobs for a full-size workload, kept in pytest's cache directory between runs
    (keyed by workload, seed and the oracle's source, written from oracle/ output only)."""
    import hashlib
    import os
    spec = batch["spec"]
    src = open(O.__file__, "rb").read()
    key = "%s_%d_%s" % (spec.name, spec.seed, hashlib.sha1(src).hexdigest()[:12])
    path = None
    if pytest_cache is not None:
        path = os.path.join(str(pytest_cache.mkdir("atgrpo_oracle")), key + ".npz")
        if os.path.exists(path):
            z = np.load(path)
            if z["lse"].shape[0] == batch["T"]:
                return z["lse"], z["logp"]
    lse, logp = oracle_logprobs(batch)
    if path is not None:
        np.savez(path, lse=lse, logp=logp)
    return lse, logp
