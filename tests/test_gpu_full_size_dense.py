"""Dense-advantage parity at the benchmark's sizes: the configuration bench.py times (qwen3_1p7b),
the three-head grouped GEMM (multi3), and the Qwen3-8B head (d = 4096, 16 d tiles, 19 vocabulary
chunks) on a quarter of its batch.

Inputs are the benchmark's batch with every response carrying its Eq. 1 advantage and old_logp
built from the ORACLE's log-probs, so the backward runs every row tile, every vocabulary chunk and
both alternating dZ buffers exactly as in the timed step: the forward keeps the logits in a lent
buffer and the backward reads them (the backward that recomputes them instead is run as well and
must give the same bits in every element of dH and dW); a third backward runs from logits kept as 16-bit
codes and is held to the same tolerances against the oracle.  The oracle computes the full forward
(lse, logp for every token; about 1e13 fp64 flop per head pass) and then, from its own lse and
gradient factors, single rows of dH and dW:
  * dH rows of tokens drawn from EVERY 128-row half of every 256-row pair tile of the backward's
    compacted row space (so both CTAs of every pair and both row blocks are sampled), plus tokens
    that carry no gradient (rows must be exactly zero);
  * dW rows of the most-hit target ids, the first and last row of every vocabulary chunk and of the
    128-row halves next to them, row 0, the last valid row V-1, and random ids.
Tolerances: logp, lse <= 1e-3 absolute for every token; loss <= 1e-3 relative; sampled gradient
blocks <= 5e-3 relative Frobenius and every sampled row within 1e-2 of its own norm (+1e-3 of the
rms row norm)."""
import numpy as np
import pytest
import torch

from oracle import atgrpo_oracle as O
from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu


def _token_sample(keep_idx, n_zero_idx, rng, per_half=3):
    """keep_idx: tokens of one head that carry a gradient, in the order the backward compacts them
    (ascending token index).  Picks per_half tokens from every 128-row half of every pair tile."""
    picks = []
    for lo in range(0, keep_idx.size, 128):
        hi = min(lo + 128, keep_idx.size)
        k = min(per_half, hi - lo)
        picks.append(keep_idx[lo + rng.choice(hi - lo, size=k, replace=False)])
        picks.append(keep_idx[[lo, hi - 1]])                   # first and last row of the half
    if n_zero_idx.size:
        picks.append(n_zero_idx[rng.choice(n_zero_idx.size, size=min(8, n_zero_idx.size), replace=False)])
    return np.unique(np.concatenate(picks))


def _vocab_sample(V, targets, n_chunks, rows_per_chunk, rng, n_random=220):
    ids = [0, V - 1]
    for c in range(n_chunks):
        lo, hi = c * rows_per_chunk, min(V, (c + 1) * rows_per_chunk)
        ids += [lo, lo + 127, lo + 128, lo + 255, lo + 256, hi - 257, hi - 129, hi - 128, hi - 1]
    top = np.argsort(-np.bincount(targets, minlength=V), kind="stable")[:48]      # most-hit target ids
    ids = np.concatenate([np.array(ids), top, rng.integers(0, V, n_random)])
    return np.unique(ids[(ids >= 0) & (ids < V)])


@pytest.mark.parametrize("name", ["qwen3_1p7b", "multi3", "qwen3_8b_quarter"])
def test_full_size_dense_backward_rows(name, request):
    b = WL.make_rollout(WL.SPECS[name])
    spec, T, M, V = b["spec"], b["T"], b["spec"].n_heads, b["spec"].V
    rng = np.random.default_rng(spec.seed + 17)
    lse, logp = U.oracle_logprobs_cached(b, request.config.cache)
    adv = U.batch_advantages(b)
    old = WL.make_old_logp(torch.from_numpy(logp), spec.seed + 100, 0.3)
    old = U.keep_off_the_kinks(logp, old)
    head, offsets, perm = U.oracle_heads(b)
    gl = torch.tensor([1.0, 0.5, 2.0][:M]) if M > 1 else None

    case = U.PolicyCase(b, adv, old, grad_loss=gl)
    case.lend_logits()                                             # as in the timed step: the forward keeps the logits
    out = case.fwd()
    assert out["status"] == 0
    assert np.array_equal(out["role_offsets"].numpy(), offsets) and np.array_equal(out["role_perm"].numpy(), perm)
    assert np.abs(out["lse"].numpy() - lse).max() <= 1e-3          # every token, not a sample
    assert np.abs(out["logp"].numpy() - logp).max() <= 1e-3
    rloss, _, rcc = O.policy_loss(logp, old, adv, b["resp_of_token"], head, M)
    np.testing.assert_allclose(out["loss"].numpy(), rloss, rtol=1e-3)
    assert np.abs(out["clip_counts"].numpy() - rcc).max() <= 2 and rcc.sum() > 100

    # the backward as timed (from the kept logits) and with the contraction recomputed: same bits
    g = case.bwd_both_ways(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    assert g["status"] == 0
    # and from logits kept as 16-bit codes (half the bytes; within the tolerances, not bit-identical)
    case.lend_logits(A.LOGITS_Q16)
    out16 = case.fwd()
    assert out16["status"] == 0 and torch.equal(out16["logp"], out["logp"]) and torch.equal(out16["lse"], out["lse"])
    g16 = case.bwd(torch.from_numpy(logp).float(), torch.from_numpy(lse).float())
    assert g16["status"] == 0
    c = O.dloss_dlogp(logp, old, adv, b["resp_of_token"], head, M, None if gl is None else gl.numpy())
    n_chunks, rows_per_chunk = A.atgrpo_policy_loss_bwd_chunks(T, spec.d, V, M)
    assert n_chunks >= 2                                           # both dZ buffers alternate
    dH = g["dH"].numpy()
    for m in range(M):
        idx = np.nonzero(head == m)[0]                             # tokens of the head, ascending
        cm = c[idx]
        keep_local = np.nonzero(cm != 0)[0]
        zero_local = np.nonzero(cm == 0)[0]
        assert keep_local.size > 256 * 3 and zero_local.size > 0
        n_halves = (keep_local.size + 127) // 128
        tok_rows = _token_sample(keep_local, zero_local, rng, per_half=max(3, -(-320 // n_halves)))
        voc_rows = _vocab_sample(V, b["target"].numpy()[idx], n_chunks, rows_per_chunk, rng)
        assert tok_rows.size >= 256 and voc_rows.size >= 256
        ref_h, ref_w = O.policy_loss_grad_rows(b["H"][idx], b["W"][m], b["target"][idx], lse[idx], cm,
                                               token_rows=tok_rows, vocab_rows=voc_rows)
        U.check_rows(dH[idx[tok_rows]], ref_h, "dH rows of head %d" % m)
        U.check_rows(g["dW"][m].numpy()[voc_rows], ref_w, "dW rows of head %d" % m)
        U.check_rows(g16["dH"].numpy()[idx[tok_rows]], ref_h, "dH rows of head %d from 16-bit codes" % m)
        U.check_rows(g16["dW"][m].numpy()[voc_rows], ref_w, "dW rows of head %d from 16-bit codes" % m)
    # every token without a gradient has an exactly zero dH row, and the identities that need no oracle
    assert (dH[c == 0] == 0).all() and (g16["dH"].numpy()[c == 0] == 0).all()
    for m in range(M):
        dW = g["dW"][m].double()
        assert dW.sum(0).abs().max().item() <= 2e-3 * dW.abs().sum(0).max().item()      # sum_v dZ_jv = 0
