#!/usr/bin/env python
"""Benchmark of the SAPO policy-scoring step (pack -> advantages -> loss forward -> backward).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 2]

Prints one JSON line.  `value` is scored tokens/s with the inputs resident in device memory;
`e2e` is the same metric with the rollout buffers starting in pinned host memory every step.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
Under torchrun every rank scores its own batch (independent replicas, no data-path
collective) and rank 0 reports the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "scored tokens/s (fwd+bwd policy loss)"
UNIT = "tokens/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": p["bf16_tflops"], "bf16_tflops_sustained": p["bf16_tflops_sustained"],
                "hbm_gbs": p["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "25"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample(batch, n_tokens_target):
    """First whole sequences of the packed batch totalling at least `n_tokens_target` tokens."""
    cu = batch.built.cu_seqlens
    s = int(np.searchsorted(cu, n_tokens_target, side="left"))
    s = max(1, min(s, batch.S))
    return s, int(cu[s])


def time_oracle(batch, n_seqs, repeats=1):
    """Seconds for the oracle to score the first n_seqs sequences (pack, advantages,
    forward, backward), as it stands."""
    from oracle import sapo_oracle as orc
    from paper_2509_08721_b200 import inputs as gen
    b = batch.built
    T = int(b.cu_seqlens[n_seqs])
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        buf = lambda x: {"hidden": x.hidden, "ids": x.ids, "old_logp": x.old_logp,
                         "offsets": x.offsets, "rewards": x.rewards}
        sel = {"q_offsets_local": batch.sel.q_offsets_local, "local_idx": batch.sel.local_idx,
               "q_offsets_ext": batch.sel.q_offsets_ext, "ext_idx": batch.sel.ext_idx}
        p = orc.pack_rollouts(buf(batch.local), buf(batch.ext), sel)
        a = orc.group_advantages(p["rewards"], p["group_offsets"])
        orc.policy_loss_fwd_bwd_rows(gen.as_f32(p["hidden"][:T]), gen.as_f32(batch.W), p["ids"][:T],
                                     p["old_logp"][:T], a["adv"][:n_seqs], p["cu_seqlens"][:n_seqs + 1],
                                     batch.eps_low, batch.eps_high, rows_per_block=512)
        times.append(time.perf_counter() - t0)
    return min(times), T


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def build_batch(workload: int, seed: int, length_div: int = 1, ext_fraction=None):
    from paper_2509_08721_b200 import inputs as gen
    recipe = gen.config(workload, length_div=length_div, ext_fraction=ext_fraction)
    if length_div != 1:
        recipe.name += f"_lengths_div{length_div}"
    return gen.make_batch(recipe, seed), recipe


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    batch, recipe = build_batch(args.workload, 1000 * args.workload, args.length_div, args.ext_fraction)
    # old log-probs: the recipe's noise around zero suffices for timing (values do not change cost)
    n_seqs, T = oracle_sample(batch, args.ref_tokens)
    for _ in range(min(args.warmup, 1)):
        time_oracle(batch, n_seqs)
    t = []
    for _ in range(args.steps):
        dt, T = time_oracle(batch, n_seqs)
        t.append(dt)
    ms = 1e3 * sum(t) / len(t)
    value = T / (ms / 1e3)
    cores = blas_threads()
    sample = f"first {n_seqs} sequences ({T} tokens) of the {batch.T}-token batch per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": recipe.name, "H": recipe.H, "V": recipe.V, "questions": recipe.Q,
                   "local_per_question": recipe.I, "external_per_question": recipe.J,
                   "tokens_per_step": T},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def hbm_kernels(torch, B, peaks, H=896, n_rollouts=2048, mean_len=288, n_groups=1 << 24):
    """Achieved HBM GB/s of the pack and advantage kernels on a scaled case (the workload-size
    launches take tens of microseconds): about 4.2 GB moved by the pack gather, 2^24 questions
    of 8 completions (1.1 GB) for the advantages, an LM-head-sized weight for Adam.  Algorithmic bytes: pack 2*T*(2H+8) (hidden row,
    id and old log-prob, read and written once), advantages 8 bytes per completion."""
    g = torch.Generator(device="cuda").manual_seed(1)
    lens = torch.randint(mean_len // 2, mean_len * 3 // 2, (2, n_rollouts), generator=g, device="cuda")
    bufs = []
    for side in range(2):
        off = torch.zeros(n_rollouts + 1, dtype=torch.int64, device="cuda")
        off[1:] = torch.cumsum(lens[side], 0)
        nt = int(off[-1].item())
        bufs.append(B.DeviceRollouts(
            torch.randn(nt, H, device="cuda", dtype=torch.bfloat16),
            torch.randint(0, 1000, (nt,), device="cuda", dtype=torch.int32),
            torch.randn(nt, device="cuda"), off, torch.rand(n_rollouts, device="cuda")))
    Q, I = n_rollouts // 4, 4                      # every question: 4 local + 4 external picks
    qo = (torch.arange(Q + 1, device="cuda", dtype=torch.int32) * I)
    perm = [torch.randperm(n_rollouts, generator=g, device="cuda").to(torch.int32) for _ in range(2)]
    sel = B.DeviceSelection(qo, perm[0], qo.clone(), perm[1])
    T = int(lens.sum().item())
    out = B.alloc_packed(T, 2 * n_rollouts, Q, H, torch.bfloat16)
    status = B.new_status()
    rewards = torch.rand(n_groups * 8, device="cuda")
    go = (torch.arange(n_groups + 1, device="cuda", dtype=torch.int32) * 8)
    adv = torch.empty_like(rewards)

    def timed(fn, iters=20, warm=3):
        for _ in range(warm):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / iters

    ms_pack = timed(lambda: B.sapo_pack_rollouts(bufs[0], bufs[1], sel, out, status))
    ms_adv = timed(lambda: B.sapo_group_advantages(rewards, go, 1e-6, 0, adv, None, None, status))
    ms_adv_warp = timed(lambda: B.sapo_group_advantages(rewards, go, 1e-6, 0, adv, None, None, status,
                                                         warp_level=True))
    assert int(status.item()) == 0 and int(out["n_tokens"].item()) == T
    # Adam step on an LM-head-sized weight: 16 bytes read + 14 written per element
    V_adam = 151936
    master = torch.randn(V_adam, H, device="cuda") * 0.02
    mom, var = torch.zeros_like(master), torch.zeros_like(master)
    grad = torch.randn(V_adam, H, device="cuda") * 1e-3
    w16 = torch.empty(V_adam, H, device="cuda", dtype=torch.bfloat16)
    ms_adam = timed(lambda: B.sapo_adam_step(master, mom, var, grad, w16, 1))
    bytes_adam = 30.0 * V_adam * H
    bytes_pack = 2.0 * T * (2 * H + 8)
    bytes_adv = 8.0 * rewards.numel() + 4.0 * n_groups
    peak = peaks["hbm_gbs"]
    mk = lambda ms, nbytes, what: {"achieved": nbytes / ms / 1e6, "peak": peak, "unit": "GB/s",
                                   "frac": nbytes / ms / 1e6 / peak, "ms": ms, "bytes": nbytes, "case": what}
    return {"pack": mk(ms_pack, bytes_pack, f"{T} tokens of {H} bf16 from {2 * n_rollouts} rollouts"),
            "advantages": mk(ms_adv, bytes_adv, f"{n_groups} questions x 8 completions, thread-per-question kernel"),
            "advantages_warp": mk(ms_adv_warp, bytes_adv, f"{n_groups} questions x 8 completions, warp-level kernel "
                                                          "(2 lanes per question; the one batches below 4096 questions take)"),
            "adam": mk(ms_adam, bytes_adam, f"weight [{V_adam}, {H}] fp32 master + moments + bf16 copy"),
            "peak_source": peaks["source"] + " (copy bandwidth)"}


# DRAM bytes per launch of the tensor-core kernels, measured with ncu on two small cases of the same
# kernels (workload 2 with lengths / 4 and / 8: 4133 and 2059 tokens, W_head still exceeds L2; a
# full-size launch holds more on the device than a capture should) and extended to the bench's
# token count as fixed + per_token * T, both from the two-point fit.  Only for hidden 896 / vocab
# 151936.  The per-token part is the panel row plus the token's hidden / output row by the
# algorithm; the forward and dz kernels are within 5 % of that, dhidden / dW_head read 10-37 % more
# (every panel tile is read by the two column tiles of its block, whose CTA pairs do not always
# share an L2 half; how often they do differs from capture to capture: 418 and 408 KB per token
# in one, 336 and 344 KB in the latest, which the table holds).  ncu_traffic() refuses an entry
# whose slope leaves the band measured for its kernel, so a kernel change cannot leave the table
# stale unnoticed.
NCU_TRAFFIC_SHAPE = (896, 151936)
NCU_TRAFFIC = {
    # kernel: (fixed bytes, bytes per token, highest slope / algorithmic ratio accepted)
    "fwd_gemm": (0.2312e9, 22.63e3, None),
    "fwd_exp": (0.2265e9, 321.1e3, 1.08),
    "bwd_dz": (0.2628e9, 302.0e3, 1.08),
    "bwd_dh": (0.2418e9, 336.2e3, 1.45),
    "bwd_dw": (0.4500e9, 344.2e3, 1.45),
}
NCU_TRAFFIC_SEPARATE = {}      # the separate calls run the same dhidden / dW_head kernels on the same panel layout


def algorithmic_bytes_per_token(kernel: str, H: int, V: int) -> float:
    vp = -(-V // 128) * 128
    return {"fwd_gemm": 2.0 * H + 12, "fwd_exp": 2.0 * vp + 2 * H, "bwd_dz": 2.0 * vp + 2 * H,
            "bwd_dh": 2.0 * vp + 4 * H, "bwd_dw": 2.0 * vp + 2 * H}[kernel]


def ncu_traffic(kernel: str, H: int, V: int, tokens_per_launch: float, separate_calls: bool = False):
    """Per-launch DRAM traffic from the ncu table, or None when there is no valid entry."""
    table = dict(NCU_TRAFFIC)
    if separate_calls:
        table.update(NCU_TRAFFIC_SEPARATE)
    if (H, V) != NCU_TRAFFIC_SHAPE or kernel not in table:
        return None
    fixed, per_token, max_ratio = table[kernel]
    alg = algorithmic_bytes_per_token(kernel, H, V)
    if max_ratio is not None and not (0.95 <= per_token / alg <= max_ratio):
        raise SystemExit(f"bench.py: the ncu traffic table for {kernel} ({per_token:.0f} B/token) no longer matches "
                         f"the kernel's algorithmic {alg:.0f} B/token: re-capture it")
    return fixed + per_token * tokens_per_launch


class Measured:
    """Device-resident and host-buffer timings of one workload."""


def measure(torch, dist, B, gen, replicas, PolicyScorer, _to_dev, args, workload, ext_fraction, steps, warmup,
            backward, rank, world, local_rank, breakdown=True, separate=True):
    """Time `steps` scoring steps of one workload: device-resident (the headline, per-kernel
    timing off), then per kernel in a short loop of its own, then from pinned host buffers, then
    (single-pass mode) the separate forward / backward calls on the same inputs."""
    m = Measured()
    batch, recipe = build_batch(workload, replicas.rank_seed(workload, rank), args.length_div, ext_fraction)
    T, S, H, V = batch.T, batch.S, batch.H, batch.V
    W = _to_dev(batch.W, "cuda")
    scorer = PolicyScorer(W, T, S, recipe.Q, eps_low=batch.eps_low, eps_high=batch.eps_high, backward=backward)

    # old log-probs = current + noise: "current" is one forward pass of the library itself
    # over the packed tokens (set-up, untimed); the noise comes from the seeded generator.
    scorer.make_host_batch(batch)
    res = scorer.step_from_host(T, S, prefetch_next=False)
    torch.cuda.synchronize()
    gen.install_old_logp(batch, res.fwd["logp"][:T].cpu().numpy())
    scorer.make_host_batch(batch)
    d = scorer._dev
    for k, t in scorer._host.items():
        d[k].copy_(t)
    view = lambda t: t.view(torch.bfloat16) if t.dtype == torch.int16 else t
    local = B.DeviceRollouts(view(d["local.hidden"]), d["local.ids"], d["local.old_logp"],
                             d["local.offsets"], d["local.rewards"])
    ext = B.DeviceRollouts(view(d["ext.hidden"]), d["ext.ids"], d["ext.old_logp"],
                           d["ext.offsets"], d["ext.rewards"])
    sel = B.DeviceSelection(d["sel.q_offsets_local"], d["sel.local_idx"], d["sel.q_offsets_ext"],
                            d["sel.ext_idx"])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, n):
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        start.record()
        for _ in range(n):
            fn()
        stop.record()
        barrier()
        ms, _ = replicas.aggregate(start.elapsed_time(stop), 0.0, device="cuda")
        return ms

    def sampled(fn, n, before=None):
        """timed(), with the clocks sampled under the same load (nvidia-smi needs a moment to
        start: the GPU is kept busy with the same steps until it reports)."""
        sampler = ClockSampler(local_rank) if rank == 0 else None
        if sampler is not None:
            t_end = time.perf_counter() + 0.5
            while time.perf_counter() < t_end:
                fn()
            torch.cuda.synchronize()
        if before is not None:
            before()
        ms = timed(fn, n)
        return ms, (sampler.stop() if sampler else None)

    dev_step = lambda: scorer.step(local, ext, sel, T, S)
    host_step = lambda: scorer.step_from_host(T, S)

    for _ in range(warmup):
        dev_step()
    torch.cuda.synchronize()
    # a library built with the cycle counters (build.py --stats, loaded through SAPO_B200_LIB) also
    # reports what its GEMM kernels counted during the headline loop
    import ctypes
    lib = B.load()
    counters = (ctypes.c_ulonglong * 48)() if hasattr(lib, "sapo_debug_wait_stats") else None
    reset = (lambda: lib.sapo_debug_wait_stats(counters, 1)) if counters is not None else None
    # 1. the headline: device-resident inputs, no per-kernel events in the stream
    m.ms_total, m.clocks = sampled(dev_step, steps, before=reset)
    scorer.check_status()
    m.kernel_cycles = None
    if counters is not None:
        torch.cuda.synchronize()
        lib.sapo_debug_wait_stats(counters, 0)
        need = 2.0 * T * V * H / (148 * 8192.0)          # tensor-pipe cycles of one contraction over all tokens
        m.kernel_cycles = {}
        for r, name in enumerate(("forward", "dz", "dhidden", "dW_head")):
            c = [int(counters[12 * r + i]) for i in range(12)]
            if c[10] == 0:
                continue
            per_step = c[10] / steps
            m.kernel_cycles[name] = {
                "launches_per_step": per_step, "sm_cycles_per_step": c[8] / steps, "us_per_step": c[9] / steps / 1e3,
                "sm_ghz": c[8] / max(1, c[9]), "tensor_pipe_cycles_needed_over_elapsed": need / (c[8] / steps),
                "mma_thread_waits_for_operands": c[1] / max(1, c[5]) if c[5] else None,
                "mma_thread_waits_for_an_accumulator": c[2] / max(1, c[5]) if c[5] else None,
                "copy_warp_waits_for_a_free_stage": c[0] / max(1, c[4]) if c[4] else None}
    # 2. the same steps with every launch bracketed by events: which kernel takes what
    m.per_kernel, m.clocks_kernels, m.kernel_steps = None, None, 0
    if breakdown:
        m.kernel_steps = max(3, min(steps, 20))
        count = {}

        def start_events():
            B.sapo_timing_enable(True)
            count["at_start"] = B.sapo_launch_count()
        _, m.clocks_kernels = sampled(dev_step, m.kernel_steps, before=start_events)
        m.launches_per_step = (B.sapo_launch_count() - count["at_start"]) / m.kernel_steps
        m.per_kernel = B.sapo_timing_read()
        B.sapo_timing_enable(False)
    else:
        launches0 = B.sapo_launch_count()
        dev_step()
        m.launches_per_step = float(B.sapo_launch_count() - launches0)
    scorer.check_status()
    # 3. end to end: the rollout buffers start in pinned host memory every step
    for _ in range(min(warmup, 3)):
        host_step()
    m.ms_e2e, m.clocks_e2e = sampled(host_step, steps)
    scorer.check_status()
    # 4. beside the single-pass call: the separate forward and backward calls (logits recomputed)
    m.separate = None
    if separate and backward == "fused":
        scorer2 = PolicyScorer(W, T, S, recipe.Q, eps_low=batch.eps_low, eps_high=batch.eps_high,
                               backward="dense")
        sep_step = lambda: scorer2.step(local, ext, sel, T, S)
        for _ in range(warmup):
            sep_step()
        n_sep = min(steps, 30)
        ms_sep, clocks_sep = sampled(sep_step, n_sep)
        scorer2.check_status()
        m.separate = (ms_sep, n_sep, clocks_sep)
        del scorer2
        torch.cuda.empty_cache()

    _, m.total_tokens = replicas.aggregate(0.0, float(T), device="cuda")
    m.steps = steps
    m.batch, m.recipe, m.scorer = batch, recipe, scorer
    # tokens with a non-zero gradient factor: the algorithmic backward work (zero-advantage groups
    # and tokens clipped on the binding side contribute nothing to either gradient);
    # t_exec = tokens the backward contractions actually run over in this mode
    g = scorer.fwd["gscale"][:T]
    m.t_act = int((g != 0).sum().item())
    if backward == "active":
        m.t_exec = int(scorer.n_active.item())
    elif backward in ("fused", "gather") and H >= 256:
        pad = (-T) % 128                 # whole 128-token blocks without any gradient are left out
        gp = torch.nn.functional.pad(g, (0, pad)).view(-1, 128)
        m.t_exec = min(T, 128 * int((gp != 0).any(dim=1).sum().item()))
    else:
        m.t_exec = T
    m.workspace_bytes = int(scorer.workspace.numel())
    return m


def summary(m, replicas, backward, peaks):
    """The short record of a workload for the `other_workloads` key."""
    b, r = m.batch, m.recipe
    T, H, V = b.T, b.H, b.V
    ms_step = m.ms_total / m.steps
    f_alg = 2.0 * T * V * H + 4.0 * m.t_act * V * H
    out = {"workload": r.name, "H": H, "V": V, "tokens_per_step": T, "active_tokens": m.t_act, "steps": m.steps,
           "backward": backward, "ms_per_step": ms_step,
           "value": replicas.throughput(m.ms_total, m.total_tokens, m.steps), "unit": UNIT,
           "e2e_value": replicas.throughput(m.ms_e2e, m.total_tokens, m.steps),
           "tflops_algorithmic": f_alg / (ms_step / 1e3) / 1e12,
           "frac_of_bf16_burst_peak_algorithmic": f_alg / (ms_step / 1e3) / 1e12 / peaks["bf16_tflops"],
           "frac_of_bf16_sustained_peak_algorithmic": f_alg / (ms_step / 1e3) / 1e12 / peaks["bf16_tflops_sustained"],
           "workspace_bytes": m.workspace_bytes, "clocks": m.clocks}
    if m.separate is not None:
        ms_sep, n_sep, _ = m.separate
        out["separate_calls_ms_per_step"] = ms_sep / n_sep
        out["separate_calls_tflops_algorithmic"] = f_alg / (ms_sep / n_sep / 1e3) / 1e12
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2509_08721_b200 import binding as B
    from paper_2509_08721_b200 import inputs as gen
    from paper_2509_08721_b200 import replicas
    from paper_2509_08721_b200.pipeline import PolicyScorer, _to_dev

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks = load_peaks()
    if args.hbm_only:            # only the bandwidth-bound kernels, on their scaled case (for profiling)
        B.load()
        if rank == 0:
            print(json.dumps({"hbm_kernels": hbm_kernels(torch, B, peaks)}))
        return 0

    mods = (torch, dist, B, gen, replicas, PolicyScorer, _to_dev)
    m = measure(*mods, args, args.workload, args.ext_fraction, args.steps, args.warmup, args.backward,
                rank, world, local_rank)
    batch, recipe, scorer = m.batch, m.recipe, m.scorer
    T, S, H, V = batch.T, batch.S, batch.H, batch.V
    ms_step = m.ms_total / args.steps
    value = replicas.throughput(m.ms_total, m.total_tokens, args.steps)
    e2e_value = replicas.throughput(m.ms_e2e, m.total_tokens, args.steps)
    h2d, d2h = scorer.h2d_bytes, scorer.d2h_bytes

    if rank == 0:
        per_kernel, ksteps = m.per_kernel, m.kernel_steps
        t_act, t_exec = m.t_act, m.t_exec
        # roofline of the dominant kernel (largest share of the per-kernel loop)
        gemm = {k: per_kernel[k] for k in ("fwd_gemm", "fwd_exp", "bwd_dz", "bwd_dh", "bwd_dw")
                if per_kernel[k]["launches"]}
        top = max(gemm, key=lambda k: gemm[k]["ms"])
        n_top = max(1, gemm[top]["launches"])
        ms_top = gemm[top]["ms"] / n_top
        per_step = n_top / ksteps                   # launches per step (one per panel chunk)
        flops_of = lambda k: 2.0 * (T if k in ("fwd_gemm", "fwd_exp") else t_exec if k == "bwd_dz" else t_act) * V * H
        achieved = flops_of(top) / per_step / (ms_top / 1e3) / 1e12
        traffic = ncu_traffic(top, H, V, T / per_step, separate_calls=args.backward not in ("fused", "gather"))
        peak = peaks["bf16_tflops_sustained"]      # the kernel is timed inside a long step
        burst = peaks["bf16_tflops"]
        # per kernel: time, and time x SM clock (median under the same load): runs under different
        # power caps compare on the second
        mhz = (m.clocks_kernels or {}).get("sm_mhz")
        kernels = {}
        for k, v in per_kernel.items():
            if not v["launches"]:
                continue
            kernels[k] = {"ms_per_step": v["ms"] / ksteps, "launches_per_step": v["launches"] / ksteps}
            if k in gemm:
                kernels[k]["tflops"] = flops_of(k) / (v["ms"] / ksteps / 1e3) / 1e12
                if mhz:
                    kernels[k]["ms_x_sm_mhz"] = v["ms"] / ksteps * mhz
                    # share of the tensor pipe's cycles the contraction needs at that clock (148 SMs x 8192 flop / cycle)
                    kernels[k]["tensor_cycles_frac_at_that_clock"] = \
                        flops_of(k) / (148 * 8192.0) / (v["ms"] / ksteps * 1e-3 * mhz * 1e6)
        gemm_ms = sum(gemm[k]["ms"] for k in gemm) / ksteps
        f_alg = 2.0 * T * V * H + 4.0 * t_act * V * H
        # the separate backward recomputes the logits (one more contraction); the fused call does not
        f_exec = 2.0 * T * V * H + (4.0 if args.backward in ("fused", "gather") else 6.0) * t_exec * V * H
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if batch.dtype == gen.DTYPE_BF16 else "f32 (split into bf16 pairs)",
            "data": "synthetic",
            "config": {"workload": recipe.name, "H": H, "V": V, "questions": recipe.Q,
                       "local_per_question": recipe.I, "external_per_question": recipe.J,
                       "tokens_per_step": T, "sequences": S, "backward": args.backward,
                       "active_tokens": t_act, "backward_tokens_executed": t_exec,
                       "workspace_bytes": m.workspace_bytes,
                       "parallelism": f"replicas x{world}",
                       "l2": "inputs larger than L2 (W_head alone is %d MB)" % (V * H * 2 // 2**20)},
            "tflops_algorithmic": f_alg / (ms_step / 1e3) / 1e12,
            "tflops_executed": f_exec / (ms_step / 1e3) / 1e12,
            "frac_of_bf16_burst_peak_algorithmic": f_alg / (ms_step / 1e3) / 1e12 / burst,
            "frac_of_bf16_burst_peak_executed": f_exec / (ms_step / 1e3) / 1e12 / burst,
            "frac_of_bf16_sustained_peak_algorithmic": f_alg / (ms_step / 1e3) / 1e12 / peak,
            "roofline": {"bound": "tensor", "kernel": top, "achieved": achieved, "peak": peak,
                         "unit": "TFLOP/s", "frac": achieved / peak, "traffic": traffic,
                         "peak_source": peaks["source"] + " (sustained bf16 GEMM; burst is %.1f)" % burst,
                         "flops_per_launch": flops_of(top) / per_step, "ms_per_launch": ms_top,
                         "all_gemm_kernels_ms_per_step": gemm_ms},
            "kernels": kernels,
            "kernels_measured": {"how": "a separate loop of %d steps with every launch bracketed by CUDA events "
                                        "(the headline loop has none)" % ksteps,
                                 "clocks": m.clocks_kernels},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": m.ms_e2e / args.steps,
                    "overlap": "every step copies its inputs from pinned host memory into one of two device "
                               "buffer sets on a copy stream; the copy for step i+1 runs while step i computes",
                    "returns": "loss and per-token log-probs go back to the host every step; dhidden and dW_head "
                               "stay in device memory, where the transformer backward and the optimiser step "
                               "read them",
                    "clocks": m.clocks_e2e},
            "gpu_launches": int(round(m.launches_per_step * args.steps)),
            "clocks": m.clocks,
        }
        if m.kernel_cycles is not None:
            line["kernel_cycles"] = {"how": "counted by the kernels themselves (clock64 and globaltimer of CTA 0, waits of "
                                            "the copy warp and the MMA thread) during the headline loop; "
                                            "8192 flop per SM and cycle",
                                     **m.kernel_cycles}
        if m.separate is not None:
            ms_sep, n_sep, clocks_sep = m.separate
            line["separate_calls"] = {
                "what": "sapo_policy_loss_fwd then sapo_policy_loss_bwd (logits recomputed), same inputs",
                "value": replicas.throughput(ms_sep, m.total_tokens, n_sep), "unit": UNIT,
                "ms_per_step": ms_sep / n_sep, "steps": n_sep,
                "tflops_algorithmic": f_alg / (ms_sep / n_sep / 1e3) / 1e12,
                "tflops_executed": (2.0 * T * V * H + 6.0 * T * V * H) / (ms_sep / n_sep / 1e3) / 1e12,
                "frac_of_bf16_burst_peak_algorithmic": f_alg / (ms_sep / n_sep / 1e3) / 1e12 / burst,
                "clocks": clocks_sep}
    del scorer, m
    torch.cuda.empty_cache()
    if world == 1 and rank == 0:
        line["hbm_kernels"] = hbm_kernels(torch, B, peaks)
        torch.cuda.empty_cache()
        if args.other_workloads and args.workload == 2 and args.length_div == 1:
            # the other bf16 workloads, a few steps each: same measurement, short record
            others = []
            for w, frac in ((3, None), (4, None), (5, 0.5)):
                mo = measure(*mods, args, w, frac, args.other_steps, 3, "fused", rank, world, local_rank,
                             breakdown=False, separate=False)
                others.append(summary(mo, replicas, "fused", peaks))
                del mo
                torch.cuda.empty_cache()
            line["other_workloads"] = others
        if not args.no_cpu_baseline:
            n_seqs, _ = oracle_sample(batch, args.ref_tokens)
            dt, Ts = time_oracle(batch, n_seqs)
            line["cpu_baseline"] = {
                "value": Ts / dt, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                "sample": f"first {n_seqs} sequences ({Ts} tokens) of the {T}-token batch, one pass, {dt:.1f} s"}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2, help="1..5; 2 is the Qwen2.5-0.5B-shaped head")
    ap.add_argument("--ref-tokens", type=int, default=None,
                    help="tokens of the bounded oracle sample (default 2048 for cpu_baseline, 512 per reference step)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--hbm-only", action="store_true",
                    help="run only the scaled pack / advantages / Adam bandwidth measurement")
    ap.add_argument("--backward", default=None, choices=["dense", "active", "fused", "gather"],
                    help="dense: forward call, then the backward call that recomputes the logits; "
                         "active: the same over the tokens whose gradient factor is non-zero only; "
                         "fused: one call that passes over the logits once (bf16 workloads; the default "
                         "for them, with the separate calls timed beside it); gather: the same call reading "
                         "the hidden states in place from the rollout buffers (the pack copies none)")
    ap.add_argument("--length-div", type=int, default=1,
                    help="divide every completion length (a small case of the same kernels for profiling)")
    ap.add_argument("--ext-fraction", type=float, default=None,
                    help="workload 5: external share J / (I + J) of every question, one of 0, 0.25, 0.5, 0.75")
    ap.add_argument("--other-workloads", dest="other_workloads", action="store_true", default=True,
                    help="after the headline (workload 2), also time workloads 3, 4 and 5 for a few steps (default)")
    ap.add_argument("--no-other-workloads", dest="other_workloads", action="store_false")
    ap.add_argument("--other-steps", type=int, default=4)
    args = ap.parse_args()
    if args.backward is None:
        args.backward = "dense" if args.workload == 1 else "fused"
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.ref_tokens is None:
        args.ref_tokens = 512 if args.impl == "reference" else 2048
    return run_reference(args) if args.impl == "reference" else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
