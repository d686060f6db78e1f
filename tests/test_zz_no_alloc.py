"""The workspace-free grouped-advantage entry point.

Some users of the library cannot allocate device memory where advantages are computed (a fixed
memory budget shared with an inference engine, a host application that owns all allocations), so
atgrpo_group_advantages_noalloc keeps its scratch in a fixed array inside the library.  That array
is shared by all calls and keeps stale contents, so the check runs two different inputs back to
back and expects every output to equal the regular entry point's bit for bit (both run the same
kernels) and to match the fp64 oracle.  The free device memory reported by the driver must not
move across a call.  This file sorts last on purpose: a run that stops at the first failure has
already run every other test."""
import pytest
import torch

from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import workloads as WL
from tests import _util as U

pytestmark = pytest.mark.gpu


def _noalloc(s, n_env, n_role, n_turn, prm=None):
    dev = U.DEV
    R, G = s["R"], n_env * n_role * n_turn
    i32, f32 = torch.int32, torch.float32
    out = dict(adv=torch.full((R,), 7.0, dtype=f32, device=dev),
               group_of_cand=torch.full((R,), -5, dtype=i32, device=dev),
               group_offsets=torch.full((G + 1,), -5, dtype=i32, device=dev),
               group_perm=torch.full((R,), -5, dtype=i32, device=dev),
               group_mean=torch.full((G,), 7.0, dtype=f32, device=dev),
               group_std=torch.full((G,), 7.0, dtype=f32, device=dev))
    status = A.new_status(dev)
    ins = [s[k].to(dev) for k in ("rewards", "env_id", "role_id", "turn_id")]
    prm = prm or A.Params()
    # a first call, not measured: the library is loaded and the scratch address looked up by now
    tiny = [t[:4].contiguous() for t in ins]
    A.atgrpo_group_advantages_noalloc(*tiny, n_env, n_role, n_turn, prm, torch.empty(4, dtype=f32, device=dev))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]              # the driver's view: sees any cudaMalloc
    before = torch.cuda.memory_allocated()
    rc = A.atgrpo_group_advantages_noalloc(*ins, n_env, n_role, n_turn, prm, device_status=status, **out)
    torch.cuda.synchronize()
    assert rc == A.OK and int(status.item()) == 0
    assert torch.cuda.memory_allocated() == before          # nothing drawn from torch's allocator
    assert torch.cuda.mem_get_info()[0] == free_before      # nothing allocated behind its back either
    res = {k: v.cpu() for k, v in out.items()}
    res["status"] = 0
    return res


def test_noalloc_matches_regular_entry_point_and_oracle_twice_in_a_row():
    # two different batches back to back: the second call sees the first call's leftovers
    first = WL.make_stress(n_env=900, n_role=4, n_turn=4, n_tokens=10, seed=21)
    second = WL.make_stress(n_env=333, n_role=3, n_turn=5, n_tokens=10, seed=22, k_max=9)
    for s, dims in ((first, (900, 4, 4)), (second, (333, 3, 5))):
        got = _noalloc(s, *dims)
        ref = U.gpu_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], *dims)
        assert ref["status"] == 0
        for k, v in got.items():
            if k != "status":
                assert torch.equal(v, ref[k]), k
        U.check_group_advantages(got, U.oracle_group_advantages(s["rewards"], s["env_id"], s["role_id"],
                                                                s["turn_id"], *dims))


def test_noalloc_at_its_documented_maximum():
    # exactly ATGRPO_NOALLOC_MAX_CAND candidates over ATGRPO_NOALLOC_MAX_GROUPS slots, bucketing
    # outputs requested: the largest scratch plan the entry point accepts
    dims = (A.NOALLOC_MAX_GROUPS // 16, 4, 4)
    s = WL.make_stress(n_env=dims[0], n_role=4, n_turn=4, n_tokens=10, seed=23, exact_R=A.NOALLOC_MAX_CAND)
    assert s["R"] == A.NOALLOC_MAX_CAND and s["G"] == A.NOALLOC_MAX_GROUPS
    got = _noalloc(s, *dims)
    ref = U.gpu_group_advantages(s["rewards"], s["env_id"], s["role_id"], s["turn_id"], *dims)
    for k, v in got.items():
        if k != "status":
            assert torch.equal(v, ref[k]), k
    U.check_group_advantages(got, U.oracle_group_advantages(s["rewards"], s["env_id"], s["role_id"],
                                                            s["turn_id"], *dims))


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch_and_bad_parameters():
    dev = U.DEV
    n = A.NOALLOC_MAX_CAND + 1
    z_f = torch.zeros(n, dtype=torch.float32, device=dev)
    z_i = torch.zeros(n, dtype=torch.int32, device=dev)
    adv = torch.full((n,), 7.0, dtype=torch.float32, device=dev)
    assert A.atgrpo_group_advantages_noalloc(z_f, z_i, z_i, z_i, 4, 1, 1, A.Params(), adv) == A.ERR_UNSUPPORTED
    small = z_f[:8], z_i[:8]
    rc = A.atgrpo_group_advantages_noalloc(small[0], small[1], small[1], small[1], A.NOALLOC_MAX_GROUPS + 1, 1, 1,
                                           A.Params(), adv[:8])
    assert rc == A.ERR_UNSUPPORTED
    # the same parameter validation as the regular entry point
    for bad in (A.Params(std_eps=float("nan")), A.Params(candidates_grouped=5), A.Params(dW_dtype=9)):
        with pytest.raises(A.AtgrpoError):
            A.atgrpo_group_advantages_noalloc(small[0], small[1], small[1], small[1], 4, 1, 1, bad, adv[:8])
    torch.cuda.synchronize()
    assert (adv == 7.0).all()                               # nothing was enqueued
