"""Pins of the fp64 oracle against things other than itself: closed forms, invariants,
brute force, finite differences and an independent library routine (torch CPU fp64
autograd / log_softmax).  Chosen so that a dropped term, a wrong sign or index, or a
transposed operand fails at least one test."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import atgrpo_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "eq1_hand_values.txt")
rng = np.random.default_rng(7)


# ----------------------------------------------------------------------------- grouping
def test_group_key_is_injective_and_dense():
    n_env, n_role, n_turn = 5, 3, 4
    seen = set()
    for e in range(n_env):
        for i in range(n_role):
            for t in range(n_turn):
                g = int(O.group_key([e], [i], [t], n_env, n_role, n_turn)[0])
                assert 0 <= g < n_env * n_role * n_turn
                seen.add(g)
    assert len(seen) == n_env * n_role * n_turn          # no collision, no hole


def test_group_key_rejects_out_of_range():
    for bad in ([4, 0, 0], [0, 2, 0], [0, 0, 3], [-1, 0, 0]):
        with pytest.raises(ValueError):
            O.group_key([bad[0]], [bad[1]], [bad[2]], 4, 2, 3)


def test_bucketing_brute_force():
    G, R = 11, 200
    key = rng.integers(0, G, R)
    key[key == 3] = 4                                   # leave slot 3 empty
    offsets, perm = O.bucket_by_key(key, G)
    assert offsets[0] == 0 and offsets[G] == R and (np.diff(offsets) >= 0).all()
    assert sorted(perm.tolist()) == list(range(R))      # bijection
    for s in range(G):                                  # O(R*G) membership, ascending order
        members = [c for c in range(R) if key[c] == s]
        assert perm[offsets[s]:offsets[s + 1]].tolist() == members
    assert offsets[4] == offsets[3]                     # the empty slot


def test_route_tokens_brute_force():
    role = rng.integers(0, 4, 300)
    sigma = np.array([1, 0, 1, 2])
    head, offsets, perm = O.route_tokens(role, sigma, 3)
    for m in range(3):
        members = [j for j in range(300) if sigma[role[j]] == m]
        assert perm[offsets[m]:offsets[m + 1]].tolist() == members
    assert (head == sigma[role]).all()


# ----------------------------------------------------------------------------- Eq. 1
def _golden_rows():
    rows = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        r, mu, sd, a = line.split("|")
        rows.append((np.array(r.split(), float), float(mu), float(sd.split()[0]),
                     np.array(a.split(), float)))
    return rows


def test_eq1_hand_values():
    eps = 1e-6
    for r, mu, sd, a in _golden_rows():
        adv, mean, std = O.group_advantages(r, np.zeros(r.size, int), 1, std_eps=eps)
        assert mean[0] == pytest.approx(mu, abs=1e-15)
        assert std[0] == pytest.approx(sd, abs=1e-15)
        np.testing.assert_allclose(adv * (1 + eps / sd), a, rtol=0, atol=1e-14)


def test_eq1_invariants_zero_mean_unit_std():
    G = 40
    sizes = rng.integers(2, 17, G)
    key = np.repeat(np.arange(G), sizes)
    r = rng.random(key.size)
    shuffle = rng.permutation(key.size)
    key, r = key[shuffle], r[shuffle]
    for ddof in (0, 1):
        adv, mean, std = O.group_advantages(r, key, G, std_eps=1e-6, ddof=ddof)
        for s in range(G):
            a = adv[key == s]
            assert abs(a.sum()) < 1e-12
            assert np.std(a, ddof=ddof) == pytest.approx(std[s] / (std[s] + 1e-6), rel=1e-12)
            assert np.std(a, ddof=ddof) == pytest.approx(1.0, abs=1e-4)
            assert mean[s] == pytest.approx(np.mean(r[key == s]), abs=1e-15)
            assert std[s] == pytest.approx(np.std(r[key == s], ddof=ddof), rel=1e-12)


def test_eq1_all_equal_and_singleton_are_exact_zero():
    r = np.array([0.3, 0.3, 0.3, 0.3, 0.7, np.float32(0.1), np.float32(0.1), np.float32(0.1)])
    key = np.array([0, 0, 0, 0, 1, 2, 2, 2])
    for ddof in (0, 1):
        adv, _, std = O.group_advantages(r, key, 4, ddof=ddof)
        assert (adv == 0.0).all()
        assert (std == 0.0).all()


def test_eq1_pair_closed_form():
    a, b, eps = 0.9, 0.25, 1e-6
    adv, _, _ = O.group_advantages([a, b], [0, 0], 1, std_eps=eps)
    want = 1.0 / (1.0 + 2 * eps / abs(a - b))
    np.testing.assert_allclose(adv, [want, -want], rtol=1e-14)
    adv1, _, _ = O.group_advantages([a, b], [0, 0], 1, std_eps=eps, ddof=1)
    sd1 = abs(a - b) / math.sqrt(2)
    np.testing.assert_allclose(adv1, [(a - b) / 2 / (sd1 + eps), -(a - b) / 2 / (sd1 + eps)], rtol=1e-14)


def test_eq1_shift_scale_and_order_invariance():
    key = np.repeat(np.arange(6), 5)
    r = rng.random(30)
    base, _, _ = O.group_advantages(r, key, 6, std_eps=0.0)
    shifted, _, _ = O.group_advantages(r + 3.0, key, 6, std_eps=0.0)
    scaled, _, _ = O.group_advantages(r * 7.0, key, 6, std_eps=0.0)
    np.testing.assert_allclose(shifted, base, atol=1e-12)
    np.testing.assert_allclose(scaled, base, atol=1e-12)
    p = rng.permutation(30)
    perm_adv, _, _ = O.group_advantages(r[p], key[p], 6, std_eps=0.0)
    np.testing.assert_allclose(perm_adv, base[p], atol=1e-15)


# ----------------------------------------------------------------------------- log-probs
def test_logp_zero_head_is_uniform():
    V = 37
    lse, logp, zt = O.token_logprobs(rng.standard_normal((5, 8)), np.zeros((V, 8)), [0, 1, 2, 3, 36])
    np.testing.assert_allclose(logp, -math.log(V), atol=1e-15)
    np.testing.assert_allclose(lse, math.log(V), atol=1e-15)


def test_logp_two_way_is_minus_softplus():
    H = rng.standard_normal((9, 6))
    W = rng.standard_normal((2, 6))
    y = rng.integers(0, 2, 9)
    _, logp, _ = O.token_logprobs(H, W, y)
    z = np.array([[h @ W[0], h @ W[1]] for h in H])
    want = [-math.log1p(math.exp(z[j, 1 - y[j]] - z[j, y[j]])) for j in range(9)]
    np.testing.assert_allclose(logp, want, atol=1e-13)


def test_logp_matches_library_log_softmax_and_is_normalised():
    T, d, V = 33, 24, 211
    H = torch.randn(T, d, dtype=torch.float64)
    W = torch.randn(V, d, dtype=torch.float64) * 3
    y = torch.randint(0, V, (T,))
    lse, logp, zt = O.token_logprobs(H.numpy(), W.numpy(), y.numpy())
    ref = torch.log_softmax(H @ W.T, dim=1)
    np.testing.assert_allclose(logp, ref[torch.arange(T), y].numpy(), atol=1e-12)
    z = (H @ W.T).numpy()
    np.testing.assert_allclose(np.exp(z - lse[:, None]).sum(1), 1.0, atol=1e-12)
    # a transposed operand or a wrong gather index would break this elementwise pin
    j = 7
    assert zt[j] == pytest.approx(sum(H[j, k].item() * W[y[j], k].item() for k in range(d)), abs=1e-12)


def test_logp_large_logits_do_not_overflow():
    H = np.full((1, 4), 100.0)
    W = np.array([[10.0] * 4, [9.0] * 4, [0.0] * 4])
    lse, logp, _ = O.token_logprobs(H, W, [0])
    assert np.isfinite(lse).all()
    assert logp[0] == pytest.approx(-math.log1p(math.exp(-400.0) + math.exp(-4000.0)), abs=1e-12)


# ----------------------------------------------------------------------------- Eq. 2
def test_loss_ratio_one_is_minus_token_mean_of_advantage():
    R, T = 6, 50
    adv = rng.standard_normal(R)
    resp = np.sort(rng.integers(0, R, T))
    logp = -rng.random(T) * 5
    loss, count, cc = O.policy_loss(logp, logp, adv, resp, np.zeros(T, int), 1)
    assert loss[0] == pytest.approx(-adv[resp].mean(), abs=1e-15)
    assert count[0] == T and (cc == 0).all()


def test_clip_branches_by_construction():
    eps = 0.2
    cases = [  # (A, ratio) -> (term, gradient passes?)
        (+2.0, 1.5, (1 + eps) * 2.0, False),     # A>0, r above the upper clip: clipped, no gradient
        (-2.0, 0.5, (1 - eps) * -2.0, False),    # A<0, r below the lower clip: clipped, no gradient
        (+2.0, 0.5, 0.5 * 2.0, True),            # A>0, r below: min picks the unclipped term
        (-2.0, 1.5, 1.5 * -2.0, True),           # A<0, r above: unclipped (no dual clip in Eq. 2)
        (+2.0, 1.1, 1.1 * 2.0, True),            # inside the trust region
        (0.0, 1.7, 0.0, False),                  # A = 0 carries nothing
    ]
    for A, r, want, passes in cases:
        term, rr, active = O.clipped_objective([math.log(r)], [0.0], [A], eps, eps)
        assert term[0] == pytest.approx(want, rel=1e-14)
        assert rr[0] == pytest.approx(r, rel=1e-14)
        assert bool(active[0]) is passes


def test_asymmetric_clip_and_wide_clip_limit():
    term, _, _ = O.clipped_objective([math.log(1.25)], [0.0], [1.0], 0.1, 0.3)
    assert term[0] == pytest.approx(1.25)
    term, _, _ = O.clipped_objective([math.log(1.25)], [0.0], [1.0], 0.3, 0.1)
    assert term[0] == pytest.approx(1.1)
    T = 40
    lp, lo, A = rng.standard_normal(T), rng.standard_normal(T), rng.standard_normal(T)
    loss, _, _ = O.policy_loss(lp, lo, A, np.arange(T), np.zeros(T, int), 1, 1e9, 1e9)
    assert loss[0] == pytest.approx(-(np.exp(lp - lo) * A).mean(), rel=1e-13)


def test_per_policy_means_and_clip_counts():
    T = 60
    head = rng.integers(0, 3, T)
    head[head == 1] = 2                                     # policy 1 owns no token
    lp, lo = -rng.random(T), -rng.random(T)
    A = rng.standard_normal(T)
    loss, count, cc = O.policy_loss(lp, lo, A, np.arange(T), head, 3)
    for m in range(3):
        sel = head == m
        one, _, c1 = O.policy_loss(lp[sel], lo[sel], A[sel], np.arange(sel.sum()), np.zeros(sel.sum(), int), 1)
        assert loss[m] == pytest.approx(one[0], abs=1e-15)
        assert (cc[m] == c1[0]).all()
    assert loss[1] == 0.0 and count[1] == 0
    r = np.exp(lp - lo)
    assert cc[:, 0].sum() == (r < 0.8).sum() and cc[:, 1].sum() == (r > 1.2).sum()


# ----------------------------------------------------------------------------- gradients
def _tiny_problem(M, T=8, d=4, V=16, seed=3):
    g = np.random.default_rng(seed)
    H = g.standard_normal((T, d))
    W = [g.standard_normal((V, d)) * 0.7 for _ in range(M)]
    y = g.integers(0, V, T)
    head = g.integers(0, M, T) if M > 1 else np.zeros(T, int)
    R = 4
    adv = g.standard_normal(R)
    adv[1] = 0.0
    resp = np.sort(g.integers(0, R, T))
    logp = np.zeros(T)
    for m in range(M):
        sel = head == m
        _, logp[sel], _ = O.token_logprobs(H[sel], W[m], y[sel])
    # ratios spread over clipped and unclipped regions, away from the kinks at 1 +- eps
    want_r = np.array([0.5, 0.9, 1.0, 1.1, 1.5, 0.7, 1.3, 1.05])[:T]
    old = logp - np.log(want_r)
    return H, W, y, head, adv, resp, old


def _scalar_loss(H, W, y, head, adv, resp, old, gl):
    M = len(W)
    logp = np.zeros(H.shape[0])
    for m in range(M):
        sel = head == m
        if sel.any():
            _, logp[sel], _ = O.token_logprobs(H[sel], W[m], y[sel])
    loss, _, _ = O.policy_loss(logp, old, adv, resp, head, M)
    return float((loss * gl).sum())


@pytest.mark.parametrize("M", [1, 2])
def test_gradients_by_central_finite_differences(M):
    H, W, y, head, adv, resp, old = _tiny_problem(M)
    gl = np.array([1.0, 0.6][:M])
    dH, dW = O.policy_loss_grads(H, W, y, old, adv, resp, head, grad_loss=gl)
    h = 1e-6
    for (j, k) in [(0, 0), (1, 2), (3, 1), (4, 3), (6, 0), (7, 2)]:
        Hp, Hm = H.copy(), H.copy()
        Hp[j, k] += h
        Hm[j, k] -= h
        fd = (_scalar_loss(Hp, W, y, head, adv, resp, old, gl) - _scalar_loss(Hm, W, y, head, adv, resp, old, gl)) / (2 * h)
        assert dH[j, k] == pytest.approx(fd, rel=1e-6, abs=1e-9)
    for m in range(M):
        for (v, k) in [(0, 0), (int(y[0]), 1), (int(y[3]), 2), (15, 3), (7, 0)]:
            Wp = [w.copy() for w in W]
            Wm_ = [w.copy() for w in W]
            Wp[m][v, k] += h
            Wm_[m][v, k] -= h
            fd = (_scalar_loss(H, Wp, y, head, adv, resp, old, gl) - _scalar_loss(H, Wm_, y, head, adv, resp, old, gl)) / (2 * h)
            assert dW[m][v, k] == pytest.approx(fd, rel=1e-6, abs=1e-9)


@pytest.mark.parametrize("M", [1, 3])
def test_gradients_match_torch_autograd(M):
    T, d, V, R = 70, 12, 90, 9
    g = torch.Generator().manual_seed(11)
    H = torch.randn(T, d, dtype=torch.float64, generator=g, requires_grad=True)
    W = [(torch.randn(V, d, dtype=torch.float64, generator=g) * 0.5).requires_grad_() for _ in range(M)]
    y = torch.randint(0, V, (T,), generator=g)
    head = torch.randint(0, M, (T,), generator=g)
    resp = torch.sort(torch.randint(0, R, (T,), generator=g)).values
    adv = torch.randn(R, dtype=torch.float64, generator=g)
    gl = torch.rand(M, dtype=torch.float64, generator=g) + 0.5
    with torch.no_grad():
        logp0 = torch.stack([torch.log_softmax(H[j] @ W[head[j]].T, 0)[y[j]] for j in range(T)])
    old = logp0 + torch.randn(T, dtype=torch.float64, generator=g) * 0.3
    # independent code path: torch autograd of the same scalar
    total = 0.0
    for m in range(M):
        sel = (head == m).nonzero().squeeze(1)
        if sel.numel() == 0:
            continue
        lp = torch.log_softmax(H[sel] @ W[m].T, 1)[torch.arange(sel.numel()), y[sel]]
        r = torch.exp(lp - old[sel])
        A = adv[resp[sel]]
        term = torch.minimum(r * A, torch.clamp(r, 0.8, 1.2) * A)
        total = total + gl[m] * (-term.mean())
    total.backward()
    dH, dW = O.policy_loss_grads(H.detach().numpy(), [w.detach().numpy() for w in W], y.numpy(),
                                 old.numpy(), adv.numpy(), resp.numpy(), head.numpy(), grad_loss=gl.numpy())
    np.testing.assert_allclose(dH, H.grad.numpy(), atol=1e-13)
    for m in range(M):
        np.testing.assert_allclose(dW[m], W[m].grad.numpy(), atol=1e-13)
    # structural identities of the gradient
    for m in range(M):
        np.testing.assert_allclose(dW[m].sum(0), 0.0, atol=1e-13)     # sum_v dz_jv = 0
    lhs = (dH * H.detach().numpy()).sum()
    rhs = sum((dW[m] * W[m].detach().numpy()).sum() for m in range(M))
    assert lhs == pytest.approx(rhs, abs=1e-12)
    # the sampled-row variant agrees with the dense one
    m = 0
    sel = (head == m).nonzero().squeeze(1).numpy()
    Hm = H.detach().numpy()[sel]
    lse, lp, _ = O.token_logprobs(Hm, W[m].detach().numpy(), y.numpy()[sel])
    c_all = O.dloss_dlogp(logp0.numpy(), old.numpy(), adv.numpy(), resp.numpy(), head.numpy(), M, gl.numpy())
    rows, vs = np.array([0, 3, len(sel) - 1]), np.array([0, int(y[sel[0]]), V - 1])
    h_rows, w_rows = O.policy_loss_grad_rows(Hm, W[m].detach().numpy(), y.numpy()[sel], lse, c_all[sel], rows, vs)
    np.testing.assert_allclose(h_rows, dH[sel][rows], atol=1e-13)
    np.testing.assert_allclose(w_rows, dW[m][vs], atol=1e-13)


def test_clipped_and_zero_advantage_tokens_have_zero_dH():
    H, W, y, head, adv, resp, old = _tiny_problem(1)
    dH, dW = O.policy_loss_grads(H, W, y, old, adv, resp, head)
    lse, logp, _ = O.token_logprobs(H, W[0], y)
    _, r, active = O.clipped_objective(logp, old, adv[resp])
    assert (~active).any() and active.any()
    assert (dH[~active] == 0.0).all()
    assert (np.abs(dH[active]).sum(1) > 0).all()


# ----------------------------------------------------------------------------- parameter update
def test_adamw_matches_torch_optimizer_over_several_steps():
    g = torch.Generator().manual_seed(5)
    theta = torch.randn(37, 11, dtype=torch.float64, generator=g)
    p = theta.clone().requires_grad_()
    opt = torch.optim.AdamW([p], lr=3e-3, betas=(0.8, 0.95), eps=1e-7, weight_decay=0.05)
    th, m, v = theta.numpy().copy(), np.zeros((37, 11)), np.zeros((37, 11))
    for step in range(1, 6):
        grad = torch.randn(37, 11, dtype=torch.float64, generator=g) * (10.0 if step == 3 else 0.1)
        total = float(grad.norm())
        p.grad = grad.clone()
        torch.nn.utils.clip_grad_norm_([p], max_norm=1.0)          # independent library routine
        opt.step()
        scale = O.clip_scale(O.grad_sumsq([grad.numpy()]), 1.0)
        assert scale == pytest.approx(min(1.0, 1.0 / (total + 1e-6)), rel=1e-12)
        th, m, v = O.adamw_step(th, m, v, grad.numpy(), step, lr=3e-3, beta1=0.8, beta2=0.95, eps=1e-7,
                                weight_decay=0.05, scale=scale)
        np.testing.assert_allclose(th, p.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_adamw_closed_forms():
    # first step from zero state: update = -lr*sign(g)/(1+eps/|g|) - lr*wd*theta
    th, m, v = O.adamw_step(np.array([2.0, -3.0]), np.zeros(2), np.zeros(2), np.array([0.5, -4.0]), 1, lr=0.1,
                            beta1=0.9, beta2=0.999, eps=0.0, weight_decay=0.1)
    np.testing.assert_allclose(th, [2.0 * 0.99 - 0.1, -3.0 * 0.99 + 0.1], rtol=1e-12)
    np.testing.assert_allclose(m, [0.05, -0.4], rtol=1e-12)
    np.testing.assert_allclose(v, [0.00025, 0.016], rtol=1e-12)
    # zero gradient: only the decoupled decay acts
    th, m, v = O.adamw_step(np.array([1.0]), np.zeros(1), np.zeros(1), np.zeros(1), 1, lr=0.5, weight_decay=0.2)
    assert th[0] == pytest.approx(0.9) and m[0] == 0 and v[0] == 0
    assert O.clip_scale(4.0, 0.0) == 1.0 and O.clip_scale(0.25, 1.0) == 1.0
    assert O.clip_scale(16.0, 1.0) == pytest.approx(1.0 / (4.0 + 1e-6))
    assert O.grad_sumsq([np.array([3.0, 4.0]), np.array([[12.0]])]) == pytest.approx(169.0)


# ----------------------------------------------------------------------------- sequence-level Eq. 2
def test_sequence_loss_reduces_to_token_loss_for_one_token_responses():
    T = 30
    lp, lo, A = -rng.random(T), -rng.random(T), rng.standard_normal(T)
    head = rng.integers(0, 2, T)
    a, ca, cca = O.policy_loss_sequence(lp, lo, A, np.arange(T), head, 2)
    b, cb, ccb = O.policy_loss(lp, lo, A, np.arange(T), head, 2)
    np.testing.assert_allclose(a, b, atol=1e-15)
    assert (ca == cb).all() and (cca == ccb).all()
    np.testing.assert_allclose(O.dloss_dlogp_sequence(lp, lo, A, np.arange(T), head, 2),
                               O.dloss_dlogp(lp, lo, A, np.arange(T), head, 2), atol=1e-15)


def test_sequence_loss_closed_forms():
    # two responses of policy 0 (3 and 2 tokens), one of policy 1; response 2 has no token
    resp = np.array([0, 0, 0, 1, 1, 3])
    head = np.array([0, 0, 0, 0, 0, 1])
    adv = np.array([2.0, -1.0, 5.0, 0.5])
    lo = np.zeros(6)
    lp = np.array([0.1, 0.2, -0.1, 0.3, 0.2, -0.05])          # r = e^0.2, e^0.5 (clipped: A<0, r>1+eps unclipped), e^-0.05
    loss, count, cc = O.policy_loss_sequence(lp, lo, adv, resp, head, 2)
    r0, r1, r3 = np.exp(0.2), np.exp(0.5), np.exp(-0.05)
    want0 = -(min(r0 * 2.0, 1.2 * 2.0) + min(r1 * -1.0, 1.2 * -1.0)) / 2
    assert loss[0] == pytest.approx(want0, rel=1e-14) and loss[1] == pytest.approx(-r3 * 0.5, rel=1e-14)
    assert count.tolist() == [2, 1] and cc.tolist() == [[0, 2], [0, 0]]
    # ratio 1 everywhere: minus the mean advantage over RESPONSES (not tokens)
    loss, _, _ = O.policy_loss_sequence(lo, lo, adv, resp, head, 2)
    assert loss[0] == pytest.approx(-(2.0 - 1.0) / 2) and loss[1] == pytest.approx(-0.5)


def test_sequence_gradients_by_finite_differences_and_autograd():
    T, d, V, R, M = 40, 6, 30, 7, 2
    g = torch.Generator().manual_seed(23)
    H = torch.randn(T, d, dtype=torch.float64, generator=g, requires_grad=True)
    W = [(torch.randn(V, d, dtype=torch.float64, generator=g) * 0.4).requires_grad_() for _ in range(M)]
    y = torch.randint(0, V, (T,), generator=g)
    resp = torch.sort(torch.randint(0, R, (T,), generator=g)).values
    role_of_resp = torch.randint(0, M, (R,), generator=g)
    head = role_of_resp[resp]
    adv = torch.randn(R, dtype=torch.float64, generator=g)
    gl = torch.tensor([1.0, 0.7], dtype=torch.float64)
    with torch.no_grad():
        logp0 = torch.stack([torch.log_softmax(H[j] @ W[head[j]].T, 0)[y[j]] for j in range(T)])
    old = logp0 + torch.randn(T, dtype=torch.float64, generator=g) * 0.08
    total = 0.0
    for m in range(M):
        terms = []
        for c in torch.unique(resp).tolist():
            sel = (resp == c).nonzero().squeeze(1)
            if head[sel[0]] != m:
                continue
            lp = torch.log_softmax(H[sel] @ W[m].T, 1)[torch.arange(sel.numel()), y[sel]]
            r = torch.exp((lp - old[sel]).sum())
            terms.append(torch.minimum(r * adv[c], torch.clamp(r, 0.8, 1.2) * adv[c]))
        if terms:
            total = total + gl[m] * (-torch.stack(terms).mean())
    total.backward()
    dH, dW = O.policy_loss_grads(H.detach().numpy(), [w.detach().numpy() for w in W], y.numpy(), old.numpy(),
                                 adv.numpy(), resp.numpy(), head.numpy(), grad_loss=gl.numpy(),
                                 reduction="sequence")
    np.testing.assert_allclose(dH, H.grad.numpy(), atol=1e-13)
    for m in range(M):
        np.testing.assert_allclose(dW[m], W[m].grad.numpy(), atol=1e-13)
    loss, _, _ = O.policy_loss_sequence(logp0.numpy(), old.numpy(), adv.numpy(), resp.numpy(), head.numpy(), M)
    assert float((torch.from_numpy(loss) * gl).sum()) == pytest.approx(float(total), rel=1e-12)


def test_group_mean_closed_form_with_unequal_group_sizes():
    # Eq. 2's E_g[(1/K) sum_c .]: group 0 has 3 candidates, group 1 has 1, group 2 (policy 1) has 2 of
    # which one has no token.  Ratio 1 everywhere, so the term of response c is just A_c.
    resp = np.array([0, 0, 1, 2, 2, 2, 3, 4, 4])             # response 5 has no token
    head = np.array([0, 0, 0, 0, 0, 0, 0, 1, 1])
    group = np.array([0, 0, 0, 1, 2, 2])
    adv = np.array([3.0, -1.0, 4.0, 10.0, 0.5, 99.0])
    z = np.zeros(9)
    loss, count, _ = O.policy_loss_sequence(z, z, adv, resp, head, 2, group_of_resp=group)
    assert loss[0] == pytest.approx(-((3.0 - 1.0 + 4.0) / 3 + 10.0) / 2, rel=1e-14)     # two groups, equal weight
    assert loss[1] == pytest.approx(-0.5, rel=1e-14)                                   # K counts responses WITH tokens
    assert count.tolist() == [2, 1]
    per_resp, _, _ = O.policy_loss_sequence(z, z, adv, resp, head, 2)
    assert per_resp[0] == pytest.approx(-(3.0 - 1.0 + 4.0 + 10.0) / 4)                 # differs: every response equal
    # equal K in every group: the two means coincide
    resp2, head2 = np.arange(6), np.zeros(6, dtype=int)
    lp, lo = -rng.random(6), -rng.random(6)
    a, _, _ = O.policy_loss_sequence(lp, lo, adv, resp2, head2, 1, group_of_resp=np.array([0, 0, 1, 1, 2, 2]))
    b, _, _ = O.policy_loss_sequence(lp, lo, adv, resp2, head2, 1)
    np.testing.assert_allclose(a, b, rtol=1e-14)
    # gradient factor: token j of response c carries -w_c * A_c * r_c (ratio 1, all unclipped)
    c = O.dloss_dlogp_sequence(z, z, adv, resp, head, 2, group_of_resp=group)
    want = -np.array([3.0 / 6, 3.0 / 6, -1.0 / 6, 4.0 / 6, 4.0 / 6, 4.0 / 6, 10.0 / 2, 0.5, 0.5])
    np.testing.assert_allclose(c, want, rtol=1e-14)


def test_group_mean_gradients_match_torch_autograd():
    T, d, V, R, M, G = 44, 6, 30, 9, 2, 4
    g = torch.Generator().manual_seed(29)
    H = torch.randn(T, d, dtype=torch.float64, generator=g, requires_grad=True)
    W = [(torch.randn(V, d, dtype=torch.float64, generator=g) * 0.4).requires_grad_() for _ in range(M)]
    y = torch.randint(0, V, (T,), generator=g)
    resp = torch.sort(torch.randint(0, R, (T,), generator=g)).values
    group = torch.tensor([0, 0, 0, 1, 2, 2, 3, 3, 3])        # group sizes 3, 1, 2, 3
    head_of_group = torch.tensor([0, 1, 0, 1])
    head = head_of_group[group][resp]
    adv = torch.randn(R, dtype=torch.float64, generator=g)
    gl = torch.tensor([1.0, 0.6], dtype=torch.float64)
    with torch.no_grad():
        logp0 = torch.stack([torch.log_softmax(H[j] @ W[head[j]].T, 0)[y[j]] for j in range(T)])
    old = logp0 + torch.randn(T, dtype=torch.float64, generator=g) * 0.08
    total = 0.0
    for m in range(M):
        per_group = []
        for q in range(G):
            if head_of_group[q] != m:
                continue
            terms = []
            for c in (group == q).nonzero().squeeze(1).tolist():
                sel = (resp == c).nonzero().squeeze(1)
                if sel.numel() == 0:
                    continue
                lp = torch.log_softmax(H[sel] @ W[m].T, 1)[torch.arange(sel.numel()), y[sel]]
                r = torch.exp((lp - old[sel]).sum())
                terms.append(torch.minimum(r * adv[c], torch.clamp(r, 0.8, 1.2) * adv[c]))
            if terms:
                per_group.append(torch.stack(terms).mean())
        total = total + gl[m] * (-torch.stack(per_group).mean())
    total.backward()
    dH, dW = O.policy_loss_grads(H.detach().numpy(), [w.detach().numpy() for w in W], y.numpy(), old.numpy(),
                                 adv.numpy(), resp.numpy(), head.numpy(), grad_loss=gl.numpy(),
                                 reduction="sequence", group_of_resp=group.numpy())
    np.testing.assert_allclose(dH, H.grad.numpy(), atol=1e-13)
    for m in range(M):
        np.testing.assert_allclose(dW[m], W[m].grad.numpy(), atol=1e-13)
    loss, _, _ = O.policy_loss_sequence(logp0.numpy(), old.numpy(), adv.numpy(), resp.numpy(), head.numpy(), M,
                                        group_of_resp=group.numpy())
    assert float((torch.from_numpy(loss) * gl).sum()) == pytest.approx(float(total.detach()), rel=1e-12)


# ----------------------------------------------------------------------------- Eq. 3 and greedy selection
def test_reward_mix_and_group_argmax():
    team = np.array([1.0, 0.0, 1.0, 0.25], dtype=np.float32)
    loc = np.array([0.5, 0.75, 0.125, 0.0], dtype=np.float32)
    np.testing.assert_array_equal(O.mix_rewards(team, loc, 1.0), [1.5, 0.75, 1.125, 0.25])
    np.testing.assert_array_equal(O.mix_rewards(team, loc, 0.5), [1.0, 0.75, 0.625, 0.125])
    np.testing.assert_array_equal(O.mix_rewards(team, loc, 0.0), loc)
    assert O.mix_rewards(team, loc).dtype == np.float32
    # argmax: brute force, ties to the lowest index, empty slot -1
    key = np.array([2, 0, 2, 0, 2, 3, 0])
    r = np.array([0.3, 0.9, 0.7, 0.9, 0.7, -1.0, 0.1])
    best = O.group_argmax(r, key, 5)
    assert best.tolist() == [1, -1, 2, 5, -1]
    for s_ in range(5):
        members = [c for c in range(7) if key[c] == s_]
        if members:
            top = max(r[c] for c in members)
            assert best[s_] == min(c for c in members if r[c] == top)
    # a constant team reward shared by a whole group cancels in Eq. 1
    k = np.repeat(np.arange(3), 4)
    loc = rng.random(12).astype(np.float32)
    team = np.repeat(np.array([0.0, 0.5, 1.0], dtype=np.float32), 4)
    a0, _, _ = O.group_advantages(O.mix_rewards(team, loc, 1.0), k, 3, std_eps=0.0)
    a1, _, _ = O.group_advantages(loc, k, 3, std_eps=0.0)
    np.testing.assert_allclose(a0, a1, atol=1e-5)
