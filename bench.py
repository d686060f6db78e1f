#!/usr/bin/env python
"""Benchmark of the AT-GRPO policy-update hot path on B200.

One step = grouped advantages (Eq. 1) -> policy loss forward through the LM head (Eq. 2) ->
backward to dH and dW, on one synthetic on-policy batch.  Default workload: the
Qwen3-1.7B-shaped single-policy head (d=2048, V=151936, ~16K response tokens).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
                  [--logits keep|recompute]

By default the forward keeps the [T, V] fp32 logits in a buffer lent to the library and the backward
reads them (a quarter less tensor work for 8 bytes of DRAM traffic per logit); --logits recompute
times the path that never writes the logits to memory and repeats the contraction in the backward.
--logits keep16 keeps them as 16-bit codes (half the bytes, no longer bit-identical to recomputing).
On one GPU the line carries the other configurations as well ("other_logits_modes").

Prints ONE JSON line (rank 0).  With --impl reference the fp64 CPU oracle is timed instead, on a
bounded token sample of the same workload.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2510_11062_b200 import workloads as WL  # noqa: E402

# DRAM bytes of the k_lm_head launches of one step come from an earlier 1-pass ncu capture, kept in
# profiles/k_lm_head_dram_traffic.json together with a digest of the kernel sources it was taken on
# (profiles/k_lm_head_qwen3_1p7b_dram_traffic.txt says how to retake it).  They are reported only
# while that digest still matches the sources: after any change to the kernel `traffic` is null.
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "k_lm_head_dram_traffic.json")
KERNEL_SOURCES = ("lm_head.cu", "sm100.cuh")


def kernel_digest():
    import hashlib
    h = hashlib.sha1()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2510_11062_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def captured_traffic(workload, mode):
    """(forward bytes, backward bytes) of one step's LM-head launches with the logits kept
    (mode "keep") or recomputed ("recompute"), or None."""
    try:
        with open(TRAFFIC_JSON) as f:
            rec = json.load(f)
    except (OSError, ValueError):
        return None
    e = rec.get("workloads", {}).get(workload, {}).get(mode)
    if e is None or rec.get("kernel_digest") != kernel_digest():
        return None
    return float(e["forward_bytes"]), float(e["backward_bytes"])


METRIC = "fused AT-GRPO loss fwd+bwd tokens/sec"
UNIT = "tokens/s"
CPU_SAMPLE_TOKENS = 2048          # cpu_baseline leg of the GPU arm: about 10 s of oracle work
REFERENCE_SAMPLE_TOKENS = 1024    # --impl reference: each step about 5 s, so 20 + 3 steps stay near two minutes


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"],
                    bf16_sustained=p["bf16_tflops_sustained"], source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------- CPU oracle leg
def oracle_sample_seconds(batch, n_tokens):
    """Times the oracle, as it stands, on the first n_tokens tokens of the batch (full vocabulary):
    advantages for the whole batch, log-probs, loss and gradients for the sample."""
    import numpy as np
    from oracle import atgrpo_oracle as O
    spec = batch["spec"]
    t0 = time.perf_counter()
    key = O.group_key(batch["env_id"], batch["role_id"], batch["turn_id"], spec.n_env, spec.n_role, spec.n_turn)
    adv, _, _ = O.group_advantages(batch["rewards"], key, spec.n_env * spec.n_role * spec.n_turn)
    sl = slice(0, n_tokens)
    if spec.n_heads > 1:
        head, _, _ = O.route_tokens(batch["role_of_token"][sl], batch["head_of_role"], spec.n_heads)
    else:
        head = np.zeros(n_tokens, dtype=np.int64)
    H, y, resp = batch["H"][sl], batch["target"][sl], batch["resp_of_token"][sl]
    logp = np.zeros(n_tokens)
    for m in range(spec.n_heads):
        sel = np.nonzero(head == m)[0]
        if sel.size:
            _, logp[sel], _ = O.token_logprobs(H[sel], batch["W"][m], y[sel])
    old = logp + 0.05 * np.sin(np.arange(n_tokens))          # any fixed perturbation
    O.policy_loss(logp, old, adv, resp, head, spec.n_heads)
    O.policy_loss_grads(H, batch["W"], y, old, adv, resp, head)
    return time.perf_counter() - t0


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count()])
    except Exception:
        return os.cpu_count()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = WL.SPECS[args.workload]
    batch = WL.make_rollout(spec)
    n = min(REFERENCE_SAMPLE_TOKENS, batch["T"])
    times = []
    for i in range(args.warmup + args.steps):
        dt = oracle_sample_seconds(batch, n)
        if i >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = n * len(times) / total
    sample = f"first {n} tokens of the batch, full vocabulary, fwd+bwd, plus advantages of all {batch['R']} candidates"
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=1, steps=args.steps, warmup=args.warmup,
                ms_per_step=1e3 * total / len(times), higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", impl="reference",
                config=dict(workload=spec.name, d=spec.d, V=spec.V, heads=spec.n_heads, tokens_per_gpu=batch["T"],
                            responses_per_gpu=batch["R"], parallelism="dp1",
                            sample="each step: the first %d tokens of the workload's batch" % n),
                cpu_baseline=dict(value=value, unit=UNIT, cores=blas_threads(), kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def mark(self):
        """The timed region starts here: samples written so far belong to the warm-up (same load)."""
        try:
            self.skip = os.path.getsize(self.tmp.name)
        except OSError:
            self.skip = 0

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        text = self.tmp.read()
        skip = getattr(self, "skip", None)
        window = "timed region" if skip is not None else "warm-up and timed calls"
        skip = skip or 0
        if skip and len(text[skip:].splitlines()) < 3:  # a short region: take the warm-up steps' samples as well
            skip, window = 0, "warm-up and timed region (same load)"
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in text[skip:].splitlines():
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[1])), smax.append(float(f[2])), power.append(float(f[3]))
            except ValueError:
                continue
            for nm, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if sm:
            out = dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), power_w_max=max(power),
                       samples=len(sm), window=window, reasons=sorted(reasons))
        return out


# ------------------------------------------------------------------------------- GPU leg
LOGITS_MODES = ("keep", "keep16", "recompute")


def logits_bytes_per_logit(mode):
    return {"keep": 4.0, "keep16": 2.125, "recompute": 0.0}[mode]


def logits_note(mode, T, V):
    if mode == "recompute":
        return "recomputed in the backward (no [T, V] buffer)"
    gb = T * ((V + 255) // 256 * 256) * logits_bytes_per_logit(mode) / 1e9
    if mode == "keep16":
        return ("kept: the forward stores [T, V] as 16-bit codes below each 32-column block's fp32 maximum in a "
                "lent buffer (%.1f GB), the backward reads it" % gb)
    return "kept: the forward stores [T, V] fp32 in a lent buffer (%.1f GB), the backward reads it" % gb


class Runner:
    """Device-resident state of one rank: inputs, outputs, workspaces; step() enqueues the path."""

    def __init__(self, batch, device, A, W=None, dW=None, accumulate=False, logits_mode="keep", logits=None):
        """W / dW: device tensors shared with other Runners (micro-batches of one update step);
        accumulate: this Runner's backward adds into dW instead of overwriting it; logits_mode: "keep" /
        "keep16" lend the library a [T, V] buffer (fp32 / 16-bit codes) so that the backward reads the
        logits instead of repeating the contraction, "recompute" does not (`logits`: such a buffer, a
        uint8 tensor shared with other Runners, large enough for each)."""
        self.A = A
        self.dev = device
        spec = self.spec = batch["spec"]
        self.T, self.R, self.M = batch["T"], batch["R"], spec.n_heads
        f32, i32 = torch.float32, torch.int32
        self.host = {k: batch[k].pin_memory() for k in
                     ("rewards", "env_id", "role_id", "turn_id", "H", "target", "resp_of_token", "role_of_token")}
        self.d = {k: v.to(device) for k, v in self.host.items()}
        self.W = W if W is not None else [w.to(device) for w in batch["W"]]
        self.head_of_role = batch["head_of_role"].to(device) if self.M > 1 else None
        self.role_of_token = self.d["role_of_token"] if self.M > 1 else None
        # the rollout generator appends the K candidates of a group together (Algorithm 1's order), so
        # the advantages take the one-pass path; the flag means nothing to the loss calls
        G = spec.n_env * spec.n_role * spec.n_turn
        T, V, dm, M = self.T, spec.V, spec.d, self.M
        self.logits, self.logits_mode = None, logits_mode
        fmt = A.LOGITS_Q16 if logits_mode == "keep16" else A.LOGITS_F32
        if logits_mode != "recompute":
            n = A.atgrpo_policy_loss_logits_bytes(T, V, fmt)
            raw = logits[:n] if logits is not None else torch.empty(n, dtype=torch.uint8, device=device)
            self.logits = raw if fmt == A.LOGITS_Q16 else raw.view(f32)
        self.prm = A.Params(accumulate_dW=1 if accumulate else 0, candidates_grouped=1, logits=self.logits,
                            logits_format=fmt)
        self.adv = torch.zeros(self.R, dtype=f32, device=device)
        self.loss = torch.zeros(M, dtype=f32, device=device)
        self.logp = torch.zeros(T, dtype=f32, device=device)
        self.lse = torch.zeros(T, dtype=f32, device=device)
        self.old_logp = torch.zeros(T, dtype=f32, device=device)
        self.dH = torch.zeros(T, dm, dtype=torch.bfloat16, device=device)
        self.dW = dW if dW is not None else [torch.zeros(V, dm, dtype=f32, device=device) for _ in range(M)]
        self.grad_loss = None
        self.status = A.new_status(device)
        self.ws_adv = A.workspace(A.atgrpo_group_advantages_workspace_bytes(self.R, G), device)
        self.ws_fwd = A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, dm, V, M, False), device)
        self.ws_bwd = A.workspace(A.atgrpo_policy_loss_workspace_bytes(T, dm, V, M, True), device)
        self.launches = 1 + A.atgrpo_policy_loss_launch_count(T, dm, V, M, False) + \
            A.atgrpo_policy_loss_launch_count(T, dm, V, M, True)
        self.host_loss = torch.zeros(M, dtype=f32).pin_memory()
        self.h2d_bytes = sum(self.host[k].numel() * self.host[k].element_size() for k in self.host
                             if k != "role_of_token" or M > 1) + T * 4
        self.host["old_logp"] = None

    def set_logits_mode(self, mode):
        """Switches how the backward obtains the logits (allocates the buffer the mode needs)."""
        A = self.A
        fmt = A.LOGITS_Q16 if mode == "keep16" else A.LOGITS_F32
        self.logits, self.logits_mode = None, mode
        if mode != "recompute":
            raw = torch.empty(A.atgrpo_policy_loss_logits_bytes(self.T, self.spec.V, fmt), dtype=torch.uint8,
                              device=self.dev)
            self.logits = raw if fmt == A.LOGITS_Q16 else raw.view(torch.float32)
        self.prm = dataclasses.replace(self.prm, logits=self.logits, logits_format=fmt)

    def drop_logits(self):
        self.logits = None
        self.prm = dataclasses.replace(self.prm, logits=None)

    def advantages(self):
        s, d = self.spec, self.d
        self.A.atgrpo_group_advantages(d["rewards"], d["env_id"], d["role_id"], d["turn_id"], s.n_env, s.n_role,
                                       s.n_turn, self.prm, self.adv, device_status=self.status, workspace=self.ws_adv)

    def forward(self):
        d = self.d
        self.A.atgrpo_policy_loss_fwd(d["H"], self.W, d["target"], self.role_of_token, self.head_of_role,
                                      d["resp_of_token"], self.adv, self.old_logp, self.prm, self.loss, self.logp,
                                      self.lse, device_status=self.status, workspace=self.ws_fwd)

    def backward(self, comm_stream=None):
        """comm_stream (multi-GPU runs): the sum of dW over the ranks runs there, chunk by chunk,
        while the main stream computes the next vocabulary chunk."""
        d = self.d
        kw = dict(H=d["H"], W=self.W, target=d["target"], role_of_token=self.role_of_token,
                  head_of_role=self.head_of_role, resp_of_token=d["resp_of_token"], adv=self.adv,
                  old_logp=self.old_logp, logp=self.logp, lse=self.lse, grad_loss=self.grad_loss,
                  params=self.prm, dH=self.dH, dW=self.dW, device_status=self.status, workspace=self.ws_bwd)
        if comm_stream is None:
            self.A.atgrpo_policy_loss_bwd(**kw)
        else:
            from paper_2510_11062_b200 import data_parallel as DP
            DP.backward_overlapped(self.A, kw, comm_stream)

    def make_old_logp(self):
        """Perf-only: old_logp = the library's own logp + N(0, 0.05) (parity runs use the oracle's)."""
        self.advantages()
        self.forward()
        torch.cuda.synchronize()
        old = WL.make_old_logp(self.logp.cpu(), self.spec.seed + 100, 0.05)
        self.host["old_logp"] = old.pin_memory()
        self.old_logp.copy_(self.host["old_logp"])

    def count_routed_rows(self):
        """Tokens whose gradient factor is non-zero: the rows the backward's three contractions run
        on (the others -- clipped ratio or zero advantage -- are skipped).  Counted once, outside any
        timed region, from the library's own factor (which tokens are non-zero does not depend on the head)."""
        coef = torch.empty(self.T, dtype=torch.float32, device=self.dev)
        loss = torch.zeros(1, dtype=torch.float32, device=self.dev)
        ws = self.A.workspace(self.A.atgrpo_clipped_loss_workspace_bytes(self.T), self.dev)
        self.A.atgrpo_clipped_loss(self.logp, self.old_logp, self.d["resp_of_token"], self.adv, self.prm, loss, coef,
                                   None, self.status, ws)
        torch.cuda.synchronize()
        self.routed_rows = int((coef != 0).sum().item())

    def make_second_input_set(self):
        """A second set of device input buffers, so that the next step's inputs can be copied from
        the host while the current step runs."""
        self.sets = [dict(d=self.d, old_logp=self.old_logp),
                     dict(d={k: torch.empty_like(v) for k, v in self.d.items()},
                          old_logp=torch.empty_like(self.old_logp))]

    def use(self, i):
        self.d, self.old_logp = self.sets[i]["d"], self.sets[i]["old_logp"]
        self.role_of_token = self.d["role_of_token"] if self.M > 1 else None

    def upload(self, i):
        """Host -> device copy of every per-step input into input set i (on the current stream)."""
        dst = self.sets[i]
        for k, v in self.host.items():
            if k == "old_logp":
                dst["old_logp"].copy_(v, non_blocking=True)
            elif k != "role_of_token" or self.M > 1:
                dst["d"][k].copy_(v, non_blocking=True)


def run_ours(args):
    from paper_2510_11062_b200 import atgrpo as A
    from paper_2510_11062_b200 import data_parallel as DP
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    A.lib()                                    # fail loudly if libatgrpo.so is missing
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    spec = WL.SPECS[args.workload]
    if world > 1:                              # weak scaling: every rank draws its own batch
        spec = WL.RolloutSpec(**{**spec.__dict__, "seed": spec.seed + 1000 * rank})
    batch = WL.make_rollout(spec)

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n = min(CPU_SAMPLE_TOKENS, batch["T"])
        dt = oracle_sample_seconds(batch, n)
        cpu_baseline = dict(value=n / dt, unit=UNIT, cores=blas_threads(), kind="oracle",
                            sample=f"first {n} tokens, full vocabulary, fwd+bwd, plus advantages of all "
                                   f"{batch['R']} candidates; {dt:.1f} s")

    r = Runner(batch, dev, A, logits_mode=args.logits)
    r.make_old_logp()
    r.count_routed_rows()
    if world > 1:
        heads = batch["head_of_role"].long()[batch["role_of_token"].long()]
        counts = torch.bincount(heads, minlength=r.M).to(dev)
        r.grad_loss, _ = DP.token_mean_scale(counts)

    comm = torch.cuda.Stream() if world > 1 else None

    def step():
        r.advantages()
        r.forward()
        r.backward(comm)

    ev = lambda: torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local) if rank == 0 else None      # started before the warm-up: nvidia-smi takes a moment to start
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()

    # ---- timed region: device-resident inputs
    marks = [[ev() for _ in range(4)] for _ in range(args.steps)]
    torch.cuda.synchronize()
    if sampler:
        sampler.mark()
    t_start, t_end = ev(), ev()
    t_start.record()
    for k in range(args.steps):
        marks[k][0].record()
        r.advantages()
        marks[k][1].record()
        r.forward()
        marks[k][2].record()
        r.backward(comm)
        marks[k][3].record()
    t_end.record()
    torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    if world > 1:
        torch.distributed.barrier()
    ms_total = t_start.elapsed_time(t_end)
    status = int(r.status.item())

    # ---- end to end: every step's inputs start in pinned host memory and are copied inside the
    # timed region, the loss is read back every step.  Two input sets: the copy of step k+1 runs on
    # a second stream while step k computes (what a training loop that prefetches its batch does).
    r.make_second_input_set()
    main, copy = torch.cuda.current_stream(), torch.cuda.Stream()

    def e2e_loop(n):
        ready, free = [ev(), ev()], [ev(), ev()]
        for f in free:
            f.record(main)
        copy.wait_stream(main)
        with torch.cuda.stream(copy):
            r.upload(0)
            ready[0].record(copy)
        for k in range(n):
            cur, nxt = k % 2, (k + 1) % 2
            if k + 1 < n:
                with torch.cuda.stream(copy):
                    copy.wait_event(free[nxt])          # the step that read set nxt has finished
                    r.upload(nxt)
                    ready[nxt].record(copy)
            main.wait_event(ready[cur])
            r.use(cur)
            step()
            r.host_loss.copy_(r.loss, non_blocking=True)
            free[cur].record(main)
        r.use(0)

    e2e_loop(2)
    torch.cuda.synchronize()
    e_start, e_end = ev(), ev()
    e_start.record()
    e2e_loop(args.steps)
    e_end.record()
    torch.cuda.synchronize()
    ms_e2e = e_start.elapsed_time(e_end)

    # ---- the same step in the other ways of obtaining the logits in the backward, each timed the same
    # way right after (3 warm-up steps, the same number of steps), so that one line carries all of them
    alts = {}
    if world == 1 and not args.main_only:
        main_prm = r.prm
        for mode in LOGITS_MODES:
            if mode == args.logits:
                continue
            r.set_logits_mode(mode)
            for _ in range(3):
                step()
            torch.cuda.synchronize()
            am = [[ev() for _ in range(3)] for _ in range(args.steps)]
            a_start, a_end = ev(), ev()
            a_start.record()
            for k in range(args.steps):
                r.advantages()
                am[k][0].record()
                r.forward()
                am[k][1].record()
                r.backward(comm)
                am[k][2].record()
            a_end.record()
            torch.cuda.synchronize()
            alts[mode] = dict(ms_total=a_start.elapsed_time(a_end),
                              fwd_ms=statistics.mean(m[0].elapsed_time(m[1]) for m in am),
                              bwd_ms=statistics.mean(m[1].elapsed_time(m[2]) for m in am))
            r.drop_logits()
        r.prm, r.logits, r.logits_mode = main_prm, main_prm.logits, args.logits

    t = torch.tensor([ms_total, ms_e2e], dtype=torch.float64, device=dev)
    tokens = torch.tensor([float(r.T)], dtype=torch.float64, device=dev)
    if world > 1:
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        torch.distributed.all_reduce(tokens)
    ms_total, ms_e2e = t.tolist()
    tokens_all = tokens.item()
    if world > 1:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()
    if rank != 0:
        return
    if status != 0:
        raise SystemExit(f"device status {status}: {A.status_string(status)}")

    adv_ms = statistics.mean(m[0].elapsed_time(m[1]) for m in marks)
    fwd_ms = statistics.mean(m[1].elapsed_time(m[2]) for m in marks)
    bwd_ms = statistics.mean(m[2].elapsed_time(m[3]) for m in marks)
    peaks = measured_peaks()
    pass_flops = 2.0 * r.T * spec.V * spec.d                  # one T x V x d contraction
    lm_s = (fwd_ms + bwd_ms) * 1e-3                           # every k_lm_head launch of a step sits in these two calls
    tf = lambda flops, sec: flops / sec / 1e12
    # The roofline is that of the STEP's dominant kernel, k_lm_head, over all its launches (one
    # forward sweep + one launch per vocabulary chunk + 1 in the backward): algorithmic work
    # 6*T*V*d (logits, dH, dW) over the forward + backward time.  Beside it: what the tensor cores
    # actually executed -- the forward on all T rows, and the backward's three contractions (logit
    # recompute, dH, dW) on the rows that carry a gradient (counted on the device, outside the
    # timed region) -- and the two calls on their own.
    algo_tf = tf(3.0 * pass_flops, lm_s)
    bwd_passes = 2.0 if r.logits is not None else 3.0         # dH, dW (+ the logits again unless they were kept)
    executed_flops = pass_flops * (1.0 + bwd_passes * r.routed_rows / max(r.T, 1))
    exec_tf = tf(executed_flops, lm_s)
    traffic = captured_traffic(spec.name, args.logits) if world == 1 else None
    n_bwd_chunks = r.A.atgrpo_policy_loss_bwd_chunks(r.T, spec.d, spec.V, r.M)[0]
    dw_elem, dh_elem = 4.0, 2.0
    kept = r.logits is not None
    bpl = logits_bytes_per_logit(args.logits)
    fwd_bytes = 2.0 * spec.d * (spec.V * spec.n_heads + r.T)                        # W and H once
    fwd_bytes += bpl * r.T * spec.V                                                 # kept logits written once
    bwd_bytes = ((bpl * r.routed_rows * spec.V if kept else 2.0 * spec.d * (spec.V * spec.n_heads + r.routed_rows))   # logits read back, or W and H once more
                 + 2.0 * spec.d * (spec.V * spec.n_heads + 2 * r.routed_rows)       # W for dH; H for dW + gather
                 + 3.0 * 2.0 * r.routed_rows * spec.V                               # dZ written once, read by dH and by dW
                 + dw_elem * spec.V * spec.d * spec.n_heads                         # dW written once
                 + 2.0 * 4.0 * r.routed_rows * spec.d * n_bwd_chunks                # fp32 dH accumulator, once per chunk
                 + dh_elem * r.T * spec.d)                                          # dH out
    value = tokens_all * args.steps / (ms_total * 1e-3)
    line = dict(
        metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=max(args.warmup, 3),
        ms_per_step=ms_total / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
        dtype="bf16", data="synthetic",
        config=dict(workload=spec.name, d=spec.d, V=spec.V, heads=spec.n_heads, tokens_per_gpu=r.T,
                    responses_per_gpu=r.R, parallelism=f"dp{world}",
                    l2="inputs larger than L2 (W alone is %.0f MB)" % (spec.V * spec.d * 2 / 1e6),
                    logits=logits_note(args.logits, r.T, spec.V),
                    old_logp="library logp + N(0,0.05) (perf-only input)"),
        gpu_launches=(r.launches) * args.steps,
        phases_ms=dict(advantages=adv_ms, forward=fwd_ms, backward=bwd_ms),
        roofline=dict(bound="tensor",
                      kernel="k_lm_head, all launches of a step (forward sweep + %d backward launches)" % (n_bwd_chunks + 1),
                      achieved=algo_tf, peak=peaks["bf16_sustained"], unit="TFLOP/s",
                      frac=algo_tf / peaks["bf16_sustained"],
                      peak_source=peaks["source"] + " sustained cuBLAS bf16 (the kernel is timed inside a long step)",
                      flops="algorithmic 6*T*V*d = %.4g per step" % (3.0 * pass_flops),
                      traffic=None if traffic is None else traffic[0] + traffic[1],
                      traffic_source="profiles/k_lm_head_dram_traffic.json (earlier ncu capture of these sources)"
                      if traffic is not None else "no capture of the current kernel sources",
                      traffic_forward=None if traffic is None else traffic[0],
                      traffic_backward=None if traffic is None else traffic[1],
                      algorithmic_bytes=fwd_bytes + bwd_bytes, algorithmic_bytes_forward=fwd_bytes,
                      algorithmic_bytes_backward=bwd_bytes,
                      executed_tflops=exec_tf, executed_frac=exec_tf / peaks["bf16_sustained"],
                      executed="forward on %d rows + %sdH, dW on the %d rows with a gradient"
                               % (r.T, "" if r.logits is not None else "recompute, ", r.routed_rows),
                      routed_rows=r.routed_rows,
                      frac_of_nominal_2250=algo_tf / 2250.0, executed_frac_of_nominal_2250=exec_tf / 2250.0,
                      forward_tflops=tf(pass_flops, fwd_ms * 1e-3),
                      forward_frac=tf(pass_flops, fwd_ms * 1e-3) / peaks["bf16_sustained"],
                      backward_algorithmic_tflops=tf(2.0 * pass_flops, bwd_ms * 1e-3),      # dH + dW
                      backward_algorithmic_frac=tf(2.0 * pass_flops, bwd_ms * 1e-3) / peaks["bf16_sustained"],
                      backward_executed_tflops=tf(3.0 * pass_flops * r.routed_rows / max(r.T, 1), bwd_ms * 1e-3),
                      backward_launches_per_call=n_bwd_chunks + 1),
        e2e=dict(value=tokens_all * args.steps / (ms_e2e * 1e-3), unit=UNIT,
                 h2d_bytes_per_step=r.h2d_bytes, d2h_bytes_per_step=r.M * 4),
        clocks=clocks, cpu_baseline=cpu_baseline)
    other = {}
    for mode, alt in alts.items():
        a_s = (alt["fwd_ms"] + alt["bwd_ms"]) * 1e-3
        a_exec = tf(pass_flops * (1.0 + (3.0 if mode == "recompute" else 2.0) * r.routed_rows / max(r.T, 1)), a_s)
        other[mode] = dict(
            logits=logits_note(mode, r.T, spec.V),
            value=r.T * args.steps / (alt["ms_total"] * 1e-3), unit=UNIT, ms_per_step=alt["ms_total"] / args.steps,
            phases_ms=dict(forward=alt["fwd_ms"], backward=alt["bwd_ms"]),
            frac=tf(3.0 * pass_flops, a_s) / peaks["bf16_sustained"], executed_tflops=a_exec,
            executed_frac=a_exec / peaks["bf16_sustained"], executed_frac_of_nominal_2250=a_exec / 2250.0)
    if other:
        line["other_logits_modes"] = dict(
            note="the same step with --logits set to the other values, each timed right after the main region "
                 "(same steps, 3 warm-up steps)", **other)
    print(json.dumps(line), flush=True)


def run_update_step(args):
    """Workload batch128: one policy update at the paper's batch scale (App. "Training Details":
    global batch 128, responses of up to 4096 tokens, gradient clipping at 1.0, Adam with lr 1e-6 and
    weight decay 0.01).  128 responses of 512-2048 tokens (T >> 100 K in total) are processed as two
    micro-batches of 64 responses each -- advantages, forward, backward -- whose dW are ACCUMULATED
    into one fp32 gradient (the second backward runs with accumulate_dW; each micro-batch weighs
    T_i / T_total so the sum is the token mean over the whole batch), followed by the gradient norm
    and one clipped AdamW step that rewrites the bf16 head.  value = tokens of the whole batch per
    second of the whole update."""
    from paper_2510_11062_b200 import atgrpo as A
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    A.lib()
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    base = WL.SPECS["long_resp"]
    n_micro = 2
    batches = [WL.make_rollout(WL.RolloutSpec(**{**base.__dict__, "seed": base.seed + 10 * i}),
                               with_weights=(i == 0)) for i in range(n_micro)]
    g = torch.Generator().manual_seed(base.seed + 99)
    for b in batches[1:]:
        b["H"] = torch.randn(b["T"], base.d, generator=g, dtype=torch.float32).to(torch.bfloat16)
        b["W"] = batches[0]["W"]
    V, dm = base.V, base.d
    W = [batches[0]["W"][0].to(dev)]
    dW = [torch.zeros(V, dm, dtype=torch.float32, device=dev)]
    keep = args.logits != "recompute"
    shared = None
    if keep:                                   # one logits buffer, sized for the larger micro-batch, used by each in turn
        fmt = A.LOGITS_Q16 if args.logits == "keep16" else A.LOGITS_F32
        shared = torch.empty(max(A.atgrpo_policy_loss_logits_bytes(b["T"], V, fmt) for b in batches),
                             dtype=torch.uint8, device=dev)
    runners = [Runner(b, dev, A, W=W, dW=dW, accumulate=(i > 0), logits_mode=args.logits, logits=shared)
               for i, b in enumerate(batches)]
    T_all = sum(r.T for r in runners)
    for r in runners:
        r.make_old_logp()
        r.count_routed_rows()
        r.grad_loss = torch.tensor([r.T / T_all], dtype=torch.float32, device=dev)
    master = W[0].float().clone()
    m1, m2 = torch.zeros_like(master), torch.zeros_like(master)
    sumsq = torch.zeros(1, dtype=torch.float64, device=dev)
    ws_n = A.workspace(A.atgrpo_grad_sumsq_workspace_bytes(), dev)
    step_no = [0]

    def step():
        for r in runners:
            r.advantages()
            r.forward()
            r.backward()
        step_no[0] += 1
        A.atgrpo_grad_sumsq(dW[0].view(-1), sumsq, ws_n)
        A.atgrpo_adamw_step(dW[0].view(-1), master.view(-1), m1.view(-1), m2.view(-1), W[0].view(-1), sumsq,
                            A.AdamWParams(step=step_no[0]))

    ev = lambda: torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)              # started before the warm-up: nvidia-smi takes a moment to start
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler.mark()
    marks = [[ev() for _ in range(3)] for _ in range(args.steps)]
    t0, t1 = ev(), ev()
    t0.record()
    for k in range(args.steps):
        marks[k][0].record()
        for r in runners:
            r.advantages()
            r.forward()
            r.backward()
        marks[k][1].record()
        step_no[0] += 1
        A.atgrpo_grad_sumsq(dW[0].view(-1), sumsq, ws_n)
        A.atgrpo_adamw_step(dW[0].view(-1), master.view(-1), m1.view(-1), m2.view(-1), W[0].view(-1), sumsq,
                            A.AdamWParams(step=step_no[0]))
        marks[k][2].record()
    t1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    for r in runners:
        st = int(r.status.item())
        if st != 0:
            raise SystemExit(f"device status {st}: {A.status_string(st)}")
    ms_total = t0.elapsed_time(t1)
    grad_ms = statistics.mean(m[0].elapsed_time(m[1]) for m in marks)
    opt_ms = statistics.mean(m[1].elapsed_time(m[2]) for m in marks)
    peaks = measured_peaks()
    algo_tf = 6.0 * T_all * V * dm / (grad_ms * 1e-3) / 1e12
    routed = sum(r.routed_rows for r in runners)
    exec_tf = 2.0 * V * dm * (T_all + (2.0 if keep else 3.0) * routed) / (grad_ms * 1e-3) / 1e12
    n_par = V * dm
    launches = sum(r.launches for r in runners) + 2
    line = dict(
        metric="AT-GRPO update step (accumulated micro-batches + clipped AdamW) tokens/sec",
        value=T_all * args.steps / (ms_total * 1e-3), unit=UNIT, n_gpus=1, steps=args.steps,
        warmup=max(args.warmup, 3), ms_per_step=ms_total / args.steps, higher_is_better=True, scaling="weak",
        vs_baseline=None, dtype="bf16", data="synthetic",
        config=dict(workload="batch128", d=dm, V=V, heads=1, responses=sum(r.R for r in runners), tokens=T_all,
                    micro_batches=[r.T for r in runners], accumulate_dW="fp32, second micro-batch adds",
                    logits=logits_note(args.logits, max(r.T for r in runners), V),
                    optimizer="grad norm + AdamW(lr 1e-6, wd 0.01, clip 1.0) on the head, bf16 head rewritten",
                    l2="inputs larger than L2", old_logp="library logp + N(0,0.05) (perf-only input)"),
        gpu_launches=launches * args.steps,
        phases_ms=dict(gradient=grad_ms, optimizer=opt_ms),
        roofline=dict(bound="tensor", kernel="k_lm_head, all launches of the update step", achieved=algo_tf,
                      peak=peaks["bf16_sustained"], unit="TFLOP/s", frac=algo_tf / peaks["bf16_sustained"],
                      peak_source=peaks["source"] + " sustained cuBLAS bf16", traffic=None,
                      executed_tflops=exec_tf, executed_frac=exec_tf / peaks["bf16_sustained"], routed_rows=routed,
                      optimizer_gbs=34.0 * n_par / (opt_ms * 1e-3) / 1e9,
                      optimizer_frac_of_hbm=34.0 * n_par / (opt_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                      optimizer_bytes="4 B (norm) + 30 B (update) per parameter"),
        clocks=clocks)
    print(json.dumps(line), flush=True)


def run_stress(args):
    """Memory-bound workload: grouped advantages over 262144 (env, role, turn) slots and the Eq. 2
    reduction over 4 Mi tokens (x scale).  L2 is flushed before every timed call (outside the
    timed events), so the GB/s are HBM figures: 20 B per candidate; 12 B per token plus 4 B per
    response for the reduction.  The *_grouped variants keep the candidates in rollout order (the
    members of a group adjacent) and set params.candidates_grouped."""
    from paper_2510_11062_b200 import atgrpo as A
    A.lib()
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    scale = 16 if args.workload.startswith("stress16") else 1
    grouped = "_grouped" in args.workload            # rollout order: the members of a group adjacent
    packed = args.workload.endswith("_packed")       # one dense group id per candidate instead of three id arrays
    s = WL.make_stress(n_env=16384 * scale, n_tokens=4_194_304 * scale, shuffle=not grouped)
    R, G, T = s["R"], s["G"], s["T"]
    d = {k: s[k].to(dev) for k in ("rewards", "env_id", "role_id", "turn_id", "group_id", "resp_of_token", "logp",
                                   "old_logp")}
    adv = torch.empty(R, device=dev)
    loss = torch.zeros(1, device=dev)
    status = A.new_status(dev)
    ws_a = A.workspace(A.atgrpo_group_advantages_workspace_bytes(R, G), dev)
    ws_l = A.workspace(A.atgrpo_clipped_loss_workspace_bytes(T), dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    prm = A.Params(candidates_grouped=1 if grouped else 0)

    def f_adv():
        if packed:
            A.atgrpo_group_advantages_packed(d["rewards"], d["group_id"], G, prm, adv, device_status=status,
                                             workspace=ws_a)
        else:
            A.atgrpo_group_advantages(d["rewards"], d["env_id"], d["role_id"], d["turn_id"], s["n_env"], s["n_role"],
                                      s["n_turn"], prm, adv, device_status=status, workspace=ws_a)

    def f_loss():
        A.atgrpo_clipped_loss(d["logp"], d["old_logp"], d["resp_of_token"], adv, prm, loss, None, None, status, ws_l)

    def timed(f):
        for _ in range(max(args.warmup, 3)):
            f()
        ts = []
        for _ in range(args.steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); f(); b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts), min(ts)

    sampler = ClockSampler(dev.index or 0)
    adv_ms, adv_best = timed(f_adv)
    loss_ms, loss_best = timed(f_loss)
    clocks = sampler.stop()
    if int(status.item()) != 0:
        raise SystemExit("device status %d" % int(status.item()))
    peaks = measured_peaks()
    cand_bytes = 12.0 if packed else 20.0           # reward + ids (one packed id, or env/role/turn) + advantage
    adv_gbs = cand_bytes * R / (adv_ms * 1e-3) / 1e9
    loss_bytes = 12.0 * T + 4.0 * R                 # logp, old_logp, response index per token; each advantage once
    loss_gbs = loss_bytes / (loss_ms * 1e-3) / 1e9
    line = dict(metric="grouped advantage HBM GB/s (%d B per candidate)" % cand_bytes, value=adv_gbs, unit="GB/s", n_gpus=1,
                steps=args.steps, warmup=max(args.warmup, 3), ms_per_step=adv_ms, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f32", data="synthetic",
                config=dict(workload=args.workload, candidates=R, group_slots=G, tokens=T,
                            candidate_order="rollout order (groups adjacent)" if grouped else "shuffled",
                            group_ids="one packed id per candidate" if packed else "env, role, turn arrays",
                            l2="flushed before every timed call"),
                gpu_launches=(1 if grouped else 4) * args.steps,
                roofline=dict(bound="hbm", kernel="k_run_advantages (one pass)" if grouped else
                              "grouped-advantage pipeline (4 launches)", achieved=adv_gbs,
                              peak=peaks["hbm_gbs"], unit="GB/s", frac=adv_gbs / peaks["hbm_gbs"], traffic=None,
                              peak_source=peaks["source"] + " copy bandwidth"),
                loss_reduction=dict(ms=loss_ms, gbs=loss_gbs, frac=loss_gbs / peaks["hbm_gbs"],
                                    bytes="12 per token + 4 per response"),
                best_ms=dict(advantages=adv_best, loss_reduction=loss_best), clocks=clocks)
    print(json.dumps(line), flush=True)


def run_adamw(args):
    """Memory-bound update of one Qwen3-1.7B-shaped head (V*d = 311 M parameters): gradient sum of
    squares + clipped AdamW step; 4 B (norm pass) + 30 B (update pass) per parameter with fp32 dW."""
    from paper_2510_11062_b200 import atgrpo as A
    A.lib()
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    n = 151936 * 2048
    g = torch.Generator(device=dev).manual_seed(1)
    grad = torch.randn(n, device=dev, generator=g) * 1e-3
    master = torch.randn(n, device=dev, generator=g) * 0.02
    m, v = torch.zeros(n, device=dev), torch.zeros(n, device=dev)
    w = torch.empty(n, dtype=torch.bfloat16, device=dev)
    sumsq = torch.zeros(1, dtype=torch.float64, device=dev)
    ws = A.workspace(A.atgrpo_grad_sumsq_workspace_bytes(), dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    t_norm, t_step = [], []
    sampler = ClockSampler(dev.index or 0)
    for i in range(max(args.warmup, 3) + args.steps):
        a, b, c = ev(), ev(), ev()
        a.record()
        A.atgrpo_grad_sumsq(grad, sumsq, ws)
        b.record()
        A.atgrpo_adamw_step(grad, master, m, v, w, sumsq, A.AdamWParams(step=i + 1))
        c.record()
        torch.cuda.synchronize()
        if i >= max(args.warmup, 3):
            t_norm.append(a.elapsed_time(b)), t_step.append(b.elapsed_time(c))
    clocks = sampler.stop()
    peaks = measured_peaks()
    ms_n, ms_s = statistics.median(t_norm), statistics.median(t_step)
    gbs = 30.0 * n / (ms_s * 1e-3) / 1e9
    line = dict(metric="AdamW head update HBM GB/s (30 B per parameter)", value=gbs, unit="GB/s", n_gpus=1,
                steps=args.steps, warmup=max(args.warmup, 3), ms_per_step=ms_n + ms_s, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f32", data="synthetic",
                config=dict(workload="adamw", parameters=n, l2="arrays larger than L2 (5.6 GB touched per step)"),
                gpu_launches=2 * args.steps,
                roofline=dict(bound="hbm", kernel="k_adamw", achieved=gbs, peak=peaks["hbm_gbs"], unit="GB/s",
                              frac=gbs / peaks["hbm_gbs"], traffic=None,
                              peak_source=peaks["source"] + " copy bandwidth"),
                grad_norm=dict(ms=ms_n, gbs=4.0 * n / (ms_n * 1e-3) / 1e9,
                               frac=4.0 * n / (ms_n * 1e-3) / 1e9 / peaks["hbm_gbs"]),
                clocks=clocks)
    print(json.dumps(line), flush=True)


def relaunch_with_ranks(args):
    """`python bench.py --gpus N` with N > 1 and no launcher around it: start N ranks of this same
    script, one per GPU, through torch.distributed.run on 127.0.0.1 (what the documented torchrun
    command does) and pass their exit code on.  Rank 0 prints the one JSON line."""
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def run_launcher_check(args):
    """--launcher-check: what a multi-rank run does around the step, with no GPU and no kernel: every
    rank joins a gloo group, draws its own batch's shape, the token counts are summed over the
    ranks and rank 0 prints one line with "value": null.  It measures nothing; it exists so that
    the rank start-up of `--gpus N` can be tested on a machine without GPUs."""
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    spec = WL.SPECS[args.workload]
    spec = WL.RolloutSpec(**{**spec.__dict__, "seed": spec.seed + 1000 * rank})
    tokens = torch.tensor([float(WL.make_rollout(spec, with_weights=False)["T"])], dtype=torch.float64)
    if world > 1:
        dist.all_reduce(tokens)
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(dict(metric=METRIC, value=None, unit=UNIT, n_gpus=world, steps=args.steps,
                              warmup=args.warmup, launcher_check=True, scaling="weak",
                              config=dict(workload=spec.name, parallelism=f"dp{world}",
                                          tokens_all_ranks=tokens.item()))), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="qwen3_1p7b", choices=sorted(WL.SPECS) + ["stress", "stress16", "stress_grouped", "stress16_grouped", "stress_grouped_packed",
                                                                     "stress16_grouped_packed", "stress_packed", "adamw", "batch128"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--logits", default="keep", choices=list(LOGITS_MODES),
                    help="keep: the forward stores the [T, V] fp32 logits in a buffer lent by the caller and the "
                         "backward reads them (same bits as recomputing); keep16: the same with 16-bit codes "
                         "(half the bytes, |logit error| <= 2^-11); recompute: the backward repeats the "
                         "contraction (no extra memory)")
    ap.add_argument("--main-only", action="store_true",
                    help="time only the --logits mode asked for, not the other ones after it (profiling runs)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--launcher-check", action="store_true",
                    help="start the ranks, join a gloo group, print a line with value null; no GPU work")
    args = ap.parse_args()
    world_env = os.environ.get("WORLD_SIZE")
    if args.gpus > 1 and world_env is None and args.impl == "ours":
        relaunch_with_ranks(args)                 # does not return
    if world_env is not None and int(world_env) != args.gpus and int(os.environ.get("RANK", "0")) == 0:
        print(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world_env}; running {world_env} ranks", file=sys.stderr)
    if args.launcher_check:
        run_launcher_check(args)
    elif args.workload == "adamw":
        run_adamw(args)
    elif args.workload == "batch128":
        run_update_step(args)
    elif args.workload.startswith("stress"):
        run_stress(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
