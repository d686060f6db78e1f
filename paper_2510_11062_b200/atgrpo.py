"""ctypes binding of libatgrpo.so: same names and arguments as include/atgrpo.h.

Only argument marshalling happens here: torch tensors supply device pointers, the current
CUDA stream and the workspace; every step of the computation runs inside the library's kernels.
There is no CPU path: loading fails loudly when the library is missing, and every compute call
requires CUDA tensors.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libatgrpo.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_BAD_INDEX, ERR_TIMEOUT, ERR_CUDA, ERR_LAYOUT = range(8)
BF16, F32 = 0, 1
REDUCE_TOKEN_MEAN, REDUCE_SEQUENCE, REDUCE_GROUP_MEAN = 0, 1, 2
LOGITS_F32, LOGITS_Q16 = 0, 1
MAX_HEADS = 8

EXPORTS = (
    "atgrpo_status_string",
    "atgrpo_group_advantages_workspace_bytes", "atgrpo_group_advantages",
    "atgrpo_group_advantages_noalloc", "atgrpo_group_advantages_packed",
    "atgrpo_group_select_workspace_bytes", "atgrpo_group_select",
    "atgrpo_clipped_loss_workspace_bytes", "atgrpo_clipped_loss",
    "atgrpo_policy_loss_workspace_bytes", "atgrpo_policy_loss_launch_count", "atgrpo_policy_loss_logits_bytes",
    "atgrpo_policy_loss_fwd", "atgrpo_policy_loss_bwd",
    "atgrpo_policy_loss_bwd_chunks", "atgrpo_policy_loss_bwd_notify",
    "atgrpo_grad_sumsq_workspace_bytes", "atgrpo_grad_sumsq", "atgrpo_adamw_step",
    "atgrpo_selftest_bounded_wait",
)


class AtgrpoError(RuntimeError):
    pass


class _Params(ctypes.Structure):
    _fields_ = [("clip_eps_low", ctypes.c_float), ("clip_eps_high", ctypes.c_float),
                ("std_eps", ctypes.c_float), ("ddof", ctypes.c_int32),
                ("dH_dtype", ctypes.c_int32), ("dW_dtype", ctypes.c_int32),
                ("accumulate_dW", ctypes.c_int32), ("reduction", ctypes.c_int32),
                ("candidates_grouped", ctypes.c_int32),
                ("group_of_resp", ctypes.c_void_p), ("group_scratch", ctypes.c_void_p),
                ("n_groups", ctypes.c_int32),
                ("logits", ctypes.c_void_p), ("logits_bytes", ctypes.c_size_t), ("logits_format", ctypes.c_int32)]


class _AdamWParams(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float),
                ("eps", ctypes.c_float), ("weight_decay", ctypes.c_float), ("max_grad_norm", ctypes.c_float),
                ("step", ctypes.c_int32)]


@dataclass
class AdamWParams:
    lr: float = 1e-6
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.01
    max_grad_norm: float = 1.0
    step: int = 1

    def c(self) -> _AdamWParams:
        return _AdamWParams(self.lr, self.beta1, self.beta2, self.eps, self.weight_decay, self.max_grad_norm,
                            self.step)


@dataclass
class Params:
    clip_eps_low: float = 0.2
    clip_eps_high: float = 0.2
    std_eps: float = 1e-6
    ddof: int = 0
    dH_dtype: int = BF16
    dW_dtype: int = F32
    accumulate_dW: int = 0
    reduction: int = 0          # REDUCE_TOKEN_MEAN, REDUCE_SEQUENCE or REDUCE_GROUP_MEAN
    candidates_grouped: int = 0  # 1: the members of every group are adjacent (checked on the device)
    group_of_resp: object = None   # REDUCE_GROUP_MEAN: int32 CUDA tensor [n_resp], group of every response
    group_scratch: object = None   # REDUCE_GROUP_MEAN: int32 CUDA tensor [n_groups], scratch owned by the caller
    logits: object = None          # policy loss: CUDA tensor of atgrpo_policy_loss_logits_bytes(T, V, logits_format) bytes, kept logits
    logits_format: int = 0         # LOGITS_F32 (the tensor is float32) or LOGITS_Q16 (the tensor is uint8)

    def c(self) -> _Params:
        n_groups = 0 if self.group_scratch is None else self.group_scratch.numel()
        g, sc = _ptr(self.group_of_resp, torch.int32), _ptr(self.group_scratch, torch.int32)
        z = _ptr(self.logits, torch.float32 if self.logits_format == LOGITS_F32 else torch.uint8)
        return _Params(self.clip_eps_low, self.clip_eps_high, self.std_eps, self.ddof,
                       self.dH_dtype, self.dW_dtype, self.accumulate_dW, self.reduction,
                       self.candidates_grouped, g.value if g else None, sc.value if sc else None, n_groups,
                       z.value if z else None,
                       0 if self.logits is None else self.logits.numel() * self.logits.element_size(), self.logits_format)


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libatgrpo.so (built by paper_2510_11062_b200.build); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise AtgrpoError(f"{LIB_PATH} not found: run `python -m paper_2510_11062_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t
        pp = ctypes.POINTER(_Params)
        L.atgrpo_status_string.restype = ctypes.c_char_p
        L.atgrpo_status_string.argtypes = [ctypes.c_int]
        L.atgrpo_group_advantages_workspace_bytes.restype = sz
        L.atgrpo_group_advantages_workspace_bytes.argtypes = [i64, i64]
        L.atgrpo_group_advantages.restype = ctypes.c_int
        L.atgrpo_group_advantages.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32, pp, vp, vp, vp, vp,
                                              vp, vp, vp, vp, sz, vp]
        L.atgrpo_group_advantages_noalloc.restype = ctypes.c_int
        L.atgrpo_group_advantages_noalloc.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32, pp, vp, vp, vp, vp,
                                                      vp, vp, vp, vp]
        L.atgrpo_group_advantages_packed.restype = ctypes.c_int
        L.atgrpo_group_advantages_packed.argtypes = [vp, vp, i64, i64, pp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.atgrpo_group_select_workspace_bytes.restype = sz
        L.atgrpo_group_select_workspace_bytes.argtypes = [i64, i64]
        L.atgrpo_group_select.restype = ctypes.c_int
        L.atgrpo_group_select.argtypes = [vp, vp, ctypes.c_float, vp, vp, vp, i64, i32, i32, i32, pp, vp, vp, vp,
                                          vp, vp, vp, vp, vp, sz, vp]
        L.atgrpo_clipped_loss_workspace_bytes.restype = sz
        L.atgrpo_clipped_loss_workspace_bytes.argtypes = [i64]
        L.atgrpo_clipped_loss.restype = ctypes.c_int
        L.atgrpo_clipped_loss.argtypes = [vp, vp, vp, vp, i64, i64, pp, vp, vp, vp, vp, vp, sz, vp]
        L.atgrpo_policy_loss_workspace_bytes.restype = sz
        L.atgrpo_policy_loss_workspace_bytes.argtypes = [i64, i32, i32, i32, i32]
        L.atgrpo_policy_loss_logits_bytes.restype = sz
        L.atgrpo_policy_loss_logits_bytes.argtypes = [i64, i32, i32]
        L.atgrpo_policy_loss_launch_count.restype = i32
        L.atgrpo_policy_loss_launch_count.argtypes = [i64, i32, i32, i32, i32]
        L.atgrpo_policy_loss_fwd.restype = ctypes.c_int
        L.atgrpo_policy_loss_fwd.argtypes = [vp, i64, ctypes.POINTER(vp), i32, vp, vp, vp, i32, vp, vp,
                                             i64, vp, i64, i32, i32, pp, vp, vp, vp, vp, vp, vp, vp,
                                             vp, sz, vp]
        L.atgrpo_policy_loss_bwd.restype = ctypes.c_int
        L.atgrpo_policy_loss_bwd.argtypes = [vp, i64, ctypes.POINTER(vp), i32, vp, vp, vp, i32, vp, vp,
                                             i64, vp, vp, vp, vp, i64, i32, i32, pp, vp,
                                             ctypes.POINTER(vp), vp, vp, sz, vp]
        L.atgrpo_policy_loss_bwd_chunks.restype = ctypes.c_int
        L.atgrpo_policy_loss_bwd_chunks.argtypes = [i64, i32, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.atgrpo_policy_loss_bwd_notify.restype = ctypes.c_int
        L.atgrpo_policy_loss_bwd_notify.argtypes = [vp, i64, ctypes.POINTER(vp), i32, vp, vp, vp, i32, vp, vp,
                                                    i64, vp, vp, vp, vp, i64, i32, i32, pp, vp,
                                                    ctypes.POINTER(vp), ctypes.POINTER(vp), i32, vp, vp, sz, vp]
        L.atgrpo_grad_sumsq_workspace_bytes.restype = sz
        L.atgrpo_grad_sumsq_workspace_bytes.argtypes = []
        L.atgrpo_grad_sumsq.restype = ctypes.c_int
        L.atgrpo_grad_sumsq.argtypes = [vp, i32, i64, vp, vp, sz, vp]
        L.atgrpo_adamw_step.restype = ctypes.c_int
        L.atgrpo_adamw_step.argtypes = [vp, i32, vp, vp, vp, vp, i64, vp, ctypes.POINTER(_AdamWParams), vp]
        L.atgrpo_selftest_bounded_wait.restype = ctypes.c_int
        L.atgrpo_selftest_bounded_wait.argtypes = [i64, vp, vp, vp]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().atgrpo_status_string(int(code)).decode()


def _check(rc: int, what: str) -> None:
    if rc != OK:
        raise AtgrpoError(f"{what}: {status_string(rc)} ({rc})")


def _ptr(t, dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise AtgrpoError("libatgrpo takes device memory only (got a CPU tensor)")
    if dtype is not None and t.dtype != dtype:
        raise AtgrpoError(f"expected {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise AtgrpoError("tensor must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr_array(tensors, dtype):
    arr = (ctypes.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = _ptr(t, dtype).value
    return arr


def new_status(device) -> torch.Tensor:
    return torch.zeros(1, dtype=torch.int32, device=device)


def workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def atgrpo_group_advantages_workspace_bytes(n_cand: int, n_groups: int) -> int:
    return int(lib().atgrpo_group_advantages_workspace_bytes(n_cand, n_groups))


def atgrpo_group_advantages(rewards, env_id, role_id, turn_id, n_env, n_role, n_turn, params: Params,
                            adv, group_of_cand=None, group_offsets=None, group_perm=None,
                            group_mean=None, group_std=None, device_status=None, workspace=None):
    """Eq. 1 over the (env, role, turn) groups; see include/atgrpo.h.  Enqueues on the current stream."""
    i32, f32 = torch.int32, torch.float32
    rc = lib().atgrpo_group_advantages(
        _ptr(rewards, f32), _ptr(env_id, i32), _ptr(role_id, i32), _ptr(turn_id, i32),
        rewards.numel(), n_env, n_role, n_turn, ctypes.byref(params.c()), _ptr(adv, f32),
        _ptr(group_of_cand, i32), _ptr(group_offsets, i32), _ptr(group_perm, i32),
        _ptr(group_mean, f32), _ptr(group_std, f32), _ptr(device_status, i32),
        _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "atgrpo_group_advantages")


def atgrpo_group_advantages_packed(rewards, group_id, n_groups, params: Params, adv, group_offsets=None,
                                   group_perm=None, group_mean=None, group_std=None, device_status=None,
                                   workspace=None):
    """Eq. 1 from one dense group id per candidate instead of the three id arrays; see include/atgrpo.h."""
    i32, f32 = torch.int32, torch.float32
    rc = lib().atgrpo_group_advantages_packed(
        _ptr(rewards, f32), _ptr(group_id, i32), rewards.numel(), n_groups, ctypes.byref(params.c()),
        _ptr(adv, f32), _ptr(group_offsets, i32), _ptr(group_perm, i32), _ptr(group_mean, f32),
        _ptr(group_std, f32), _ptr(device_status, i32), _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "atgrpo_group_advantages_packed")


NOALLOC_MAX_CAND, NOALLOC_MAX_GROUPS = 262144, 65536


def atgrpo_group_advantages_noalloc(rewards, env_id, role_id, turn_id, n_env, n_role, n_turn, params: Params,
                                    adv, group_of_cand=None, group_offsets=None, group_perm=None,
                                    group_mean=None, group_std=None, device_status=None):
    """atgrpo_group_advantages for callers that may not allocate device memory: no workspace
    argument, the scratch is a fixed array inside the library (see include/atgrpo.h for the size
    limits and the sharing rules).  Returns the status code instead of raising on
    ERR_UNSUPPORTED so callers can fall back when a batch is too large."""
    i32, f32 = torch.int32, torch.float32
    rc = lib().atgrpo_group_advantages_noalloc(
        _ptr(rewards, f32), _ptr(env_id, i32), _ptr(role_id, i32), _ptr(turn_id, i32),
        rewards.numel(), n_env, n_role, n_turn, ctypes.byref(params.c()), _ptr(adv, f32),
        _ptr(group_of_cand, i32), _ptr(group_offsets, i32), _ptr(group_perm, i32),
        _ptr(group_mean, f32), _ptr(group_std, f32), _ptr(device_status, i32), _stream())
    if rc != ERR_UNSUPPORTED:
        _check(rc, "atgrpo_group_advantages_noalloc")
    return rc


def atgrpo_group_select_workspace_bytes(n_cand: int, n_groups: int) -> int:
    return int(lib().atgrpo_group_select_workspace_bytes(n_cand, n_groups))


def atgrpo_group_select(r_team, r_loc, alpha, env_id, role_id, turn_id, n_env, n_role, n_turn, params: Params,
                        adv, rewards_out=None, group_best=None, group_of_cand=None, group_mean=None,
                        group_std=None, device_status=None, workspace=None):
    """Eq. 3 mix + Eq. 1 advantages + per-group greedy argmax in one call; see include/atgrpo.h."""
    i32, f32 = torch.int32, torch.float32
    rc = lib().atgrpo_group_select(
        _ptr(r_team, f32), _ptr(r_loc, f32), float(alpha), _ptr(env_id, i32), _ptr(role_id, i32),
        _ptr(turn_id, i32), r_team.numel(), n_env, n_role, n_turn, ctypes.byref(params.c()),
        _ptr(rewards_out, f32), _ptr(adv, f32), _ptr(group_best, i32), _ptr(group_of_cand, i32),
        _ptr(group_mean, f32), _ptr(group_std, f32), _ptr(device_status, i32), _ptr(workspace),
        workspace.numel(), _stream())
    _check(rc, "atgrpo_group_select")


def atgrpo_clipped_loss_workspace_bytes(T: int) -> int:
    return int(lib().atgrpo_clipped_loss_workspace_bytes(T))


def atgrpo_clipped_loss(logp, old_logp, resp_of_token, adv, params: Params, loss, coef=None,
                        clip_counts=None, device_status=None, workspace=None):
    """Eq. 2 from given log-probabilities (one policy); see include/atgrpo.h."""
    i32, f32 = torch.int32, torch.float32
    rc = lib().atgrpo_clipped_loss(
        _ptr(logp, f32), _ptr(old_logp, f32), _ptr(resp_of_token, i32), _ptr(adv, f32),
        logp.numel(), adv.numel(), ctypes.byref(params.c()), _ptr(loss, f32), _ptr(coef, f32),
        _ptr(clip_counts, torch.int64), _ptr(device_status, i32), _ptr(workspace),
        workspace.numel(), _stream())
    _check(rc, "atgrpo_clipped_loss")


def atgrpo_policy_loss_workspace_bytes(T: int, d: int, V: int, M: int, is_bwd: bool) -> int:
    return int(lib().atgrpo_policy_loss_workspace_bytes(T, d, V, M, 1 if is_bwd else 0))


def atgrpo_policy_loss_logits_bytes(T: int, V: int, logits_format: int = LOGITS_F32) -> int:
    return int(lib().atgrpo_policy_loss_logits_bytes(T, V, logits_format))


def atgrpo_policy_loss_launch_count(T: int, d: int, V: int, M: int, is_bwd: bool) -> int:
    return int(lib().atgrpo_policy_loss_launch_count(T, d, V, M, 1 if is_bwd else 0))


def atgrpo_policy_loss_fwd(H, W, target, role_of_token, head_of_role, resp_of_token, adv, old_logp,
                           params: Params, loss, logp, lse, role_offsets=None, role_perm=None,
                           clip_counts=None, device_status=None, workspace=None):
    """Eq. 2 through the LM head(s) W (list of [V,d] bf16 tensors), forward; see include/atgrpo.h."""
    i32, f32, bf = torch.int32, torch.float32, torch.bfloat16
    T, d = H.shape
    V = W[0].shape[0]
    if H.stride(1) != 1:
        raise AtgrpoError("H must have unit stride along d")
    n_role = 0 if head_of_role is None else head_of_role.numel()
    rc = lib().atgrpo_policy_loss_fwd(
        ctypes.c_void_p(H.data_ptr()), H.stride(0) if T > 1 else d, _ptr_array(W, bf), len(W),
        _ptr(target, i32), _ptr(role_of_token, i32), _ptr(head_of_role, i32), n_role,
        _ptr(resp_of_token, i32), _ptr(adv, f32), adv.numel(), _ptr(old_logp, f32), T, d, V,
        ctypes.byref(params.c()), _ptr(loss, f32), _ptr(logp, f32), _ptr(lse, f32),
        _ptr(role_offsets, i32), _ptr(role_perm, i32), _ptr(clip_counts, torch.int64),
        _ptr(device_status, i32), _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "atgrpo_policy_loss_fwd")


def atgrpo_policy_loss_bwd_chunks(T: int, d: int, V: int, M: int):
    """(n_chunks, rows_per_chunk) of the vocabulary walk of one backward call; see include/atgrpo.h."""
    n, rows = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(lib().atgrpo_policy_loss_bwd_chunks(T, d, V, M, ctypes.byref(n), ctypes.byref(rows)),
           "atgrpo_policy_loss_bwd_chunks")
    return n.value, rows.value


def atgrpo_policy_loss_bwd(H, W, target, role_of_token, head_of_role, resp_of_token, adv, old_logp,
                           logp, lse, grad_loss, params: Params, dH, dW, device_status=None,
                           workspace=None, chunk_events=None):
    """Gradient of sum_m grad_loss[m]*loss[m] w.r.t. H and every W_m; see include/atgrpo.h.
    With chunk_events (a list of torch.cuda.Event, one per vocabulary chunk) the call goes through
    atgrpo_policy_loss_bwd_notify: event c is recorded when the dW rows of chunk c are final."""
    i32, f32, bf = torch.int32, torch.float32, torch.bfloat16
    T, d = H.shape
    V = W[0].shape[0]
    n_role = 0 if head_of_role is None else head_of_role.numel()
    dh_t = bf if params.dH_dtype == BF16 else f32
    dw_t = bf if params.dW_dtype == BF16 else f32
    head = (ctypes.c_void_p(H.data_ptr()), H.stride(0) if T > 1 else d, _ptr_array(W, bf), len(W),
            _ptr(target, i32), _ptr(role_of_token, i32), _ptr(head_of_role, i32), n_role,
            _ptr(resp_of_token, i32), _ptr(adv, f32), adv.numel(), _ptr(old_logp, f32),
            _ptr(logp, f32), _ptr(lse, f32), _ptr(grad_loss, f32), T, d, V, ctypes.byref(params.c()),
            _ptr(dH, dh_t), _ptr_array(dW, dw_t))
    tail = (_ptr(device_status, i32), _ptr(workspace), workspace.numel(), _stream())
    if chunk_events is None:
        rc = lib().atgrpo_policy_loss_bwd(*head, *tail)
        _check(rc, "atgrpo_policy_loss_bwd")
        return
    handles = []
    for ev in chunk_events:
        if not ev.cuda_event:            # torch creates the CUDA event on its first record
            ev.record()
        handles.append(ev.cuda_event)
    arr = (ctypes.c_void_p * len(handles))(*handles)
    rc = lib().atgrpo_policy_loss_bwd_notify(*head, arr, len(handles), *tail)
    _check(rc, "atgrpo_policy_loss_bwd_notify")


def atgrpo_grad_sumsq_workspace_bytes() -> int:
    return int(lib().atgrpo_grad_sumsq_workspace_bytes())


def atgrpo_grad_sumsq(grad, sumsq, workspace):
    """sumsq[0] (float64, device) = sum of squares of `grad` (fp32 or bf16); see include/atgrpo.h."""
    dt = BF16 if grad.dtype == torch.bfloat16 else F32
    rc = lib().atgrpo_grad_sumsq(_ptr(grad), dt, grad.numel(), _ptr(sumsq, torch.float64), _ptr(workspace),
                                 workspace.numel(), _stream())
    _check(rc, "atgrpo_grad_sumsq")


def atgrpo_adamw_step(grad, master, m, v, w_bf16, grad_sumsq, params: AdamWParams):
    """Clipped AdamW step on one head, in place on master / m / v; see include/atgrpo.h."""
    f32 = torch.float32
    dt = BF16 if grad.dtype == torch.bfloat16 else F32
    rc = lib().atgrpo_adamw_step(_ptr(grad), dt, _ptr(master, f32), _ptr(m, f32), _ptr(v, f32),
                                 _ptr(w_bf16, torch.bfloat16), master.numel(),
                                 _ptr(grad_sumsq, torch.float64), ctypes.byref(params.c()), _stream())
    _check(rc, "atgrpo_adamw_step")


def atgrpo_selftest_bounded_wait(limit_ns: int, device_status, waited=None) -> int:
    """Runs the bounded-wait self-test kernel (see include/atgrpo.h); returns the host status code."""
    i32 = torch.int32
    return int(lib().atgrpo_selftest_bounded_wait(int(limit_ns), _ptr(device_status, i32), _ptr(waited, i32),
                                                  _stream()))
