#!/usr/bin/env python
"""Benchmark of the PPO learner step (TrainPPO over an on-device rollout buffer) on B200.

One "step" is one pass of the whole hot path over one buffer of synthetic rollouts:
GAE + advantage normalisation, then for every epoch and minibatch the permutation gather,
encoder forward, fused loss, encoder backward and Adam.  The metric is env-steps trained
per second = M * epochs / time, with the buffer resident in HBM (`value`) and with the
rollout arriving from pinned host memory every step (`e2e`).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

The default workload is the largest single-GPU configuration (cfg4: 8192 envs x 16 steps of 320x240 depth).

With N > 1 (torchrun) every rank trains an independent replica on its own buffer: the
path has no exchange step on one learner GPU, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the encoder kernels of one forward + backward per
# sample row, from ncu captures of small twins of the workloads (traffic grows in proportion to the rows): workload
# -> (bytes per row, capture).  An entry is dropped (traffic: null) as soon as a kernel it covers changes.
NCU_DRAM_BYTES_PER_ROW = {
    "cfg2": (2.7490e6, "ncu capture of cfg2_prof at 512 rows, scaled by rows: profiles/ncu_main_kernels_cfg2_prof.md"),
    "cfg3": (2.7490e6, "ncu capture of cfg2_prof at 512 rows, scaled by rows: profiles/ncu_main_kernels_cfg2_prof.md"),
    "cfg2_prof": (2.7490e6, "ncu capture of cfg2_prof at 512 rows: profiles/ncu_main_kernels_cfg2_prof.md"),
    "cfg4": (11.4461e6, "ncu capture of cfg4_prof at 128 rows, scaled by rows: profiles/ncu_main_kernels_cfg4_prof.md"),
    "cfg4_prof": (11.4461e6, "ncu capture of cfg4_prof at 128 rows: profiles/ncu_main_kernels_cfg4_prof.md"),
}
METRIC = "ppo_learner_env_steps_trained_per_sec"
UNIT = "env-steps/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------- work model ----

def conv_dims(w):
    hs, ws, cs = [w.H], [w.W], [1]
    for c, k in zip(w.conv_c, w.conv_k):
        hs.append((hs[-1] + 2 * (k // 2) - k) // 2 + 1)
        ws.append((ws[-1] + 2 * (k // 2) - k) // 2 + 1)
        cs.append(c)
    return hs, ws, cs


def fwd_flops_per_sample(w, skip_conv1=False):
    """Algorithmic flops of the network's own MACs (2 * Cout * Ho * Wo * Cin * k^2 per conv, 2 * in * out per FC)."""
    hs, ws, cs = conv_dims(w)
    f = 0
    for l, k in enumerate(w.conv_k):
        if skip_conv1 and l == 0:
            continue
        f += 2 * cs[l + 1] * hs[l + 1] * ws[l + 1] * cs[l] * k * k
    i = cs[-1] + w.P
    if getattr(w, "embed", 0):
        f += 2 * hs[-1] * ws[-1] * cs[-1] * w.embed
        i = w.embed + w.P
    for _ in range(getattr(w, "n_lstm", 0)):  # W_x x and W_h h_prev of the four gates
        f += 2 * 4 * w.lstm_h * (i + w.lstm_h)
        i = w.lstm_h
    for o in list(w.fc) + [w.A + 1]:
        f += 2 * i * o
        i = o
    return f


def bwd_flops_per_sample(w):
    """dgrad + wgrad = 2x the forward for every layer except conv1, which has no dgrad."""
    hs, ws, cs = conv_dims(w)
    conv1 = 2 * cs[1] * hs[1] * ws[1] * w.conv_k[0] ** 2
    return 2 * fwd_flops_per_sample(w) - conv1


def record_bytes(w):
    return w.H * w.W * 2 + w.P * 4 + w.A * 4 + 4 * 4


# --------------------------------------------------------------------- clocks ----

class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.idx = device_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [r.split(",") for r in open(self.f.name).read().strip().splitlines() if r.count(",") >= 8]
        os.unlink(self.f.name)
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = sorted(float(r[1]) for r in rows)
        reasons = set()
        for r in rows:
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7),
                              ("sw_power_cap", 8)):
                if r[col].strip().lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(rows[0][2]), "samples": len(rows),
                "power_w_max": max(float(r[3]) for r in rows), "reasons": sorted(reasons)}


# ------------------------------------------------------------------ our arm ------

def make_learner(w, microbatch, device):
    """Seeded parameters, a device-generated rollout, actions/log-probs from the rollout policy, buffer filled."""
    import torch
    from paper_2509_16434_b200 import synth
    from paper_2509_16434_b200.learner import Learner
    L = Learner(w, microbatch, device)
    offs = L.model.tensors()
    shapes, gammas = synth.param_shapes(w)
    theta = synth.init_params(L.model.arena, [o for o, _ in offs], shapes, w.seed, ones=gammas)
    L.model.load(theta)
    roll = synth.rollout_torch(w, device, w.seed)
    action = torch.empty((w.T, w.N, w.A), dtype=torch.float32, device=device)
    logp = torch.empty((w.T, w.N), dtype=torch.float32, device=device)
    for t in range(w.T):
        a, lp, _ = L.act(roll["depth"][t], roll["proprio"][t], roll["eps"][t])
        action[t], logp[t] = a, lp
    # jitter the old log-probs so that both branches of the clip do work, as after the first update of an epoch
    logp += roll["logp_jitter"]
    roll["action"], roll["logp"] = action, logp
    L.write_rollout(roll, action, logp)
    torch.cuda.synchronize()
    return L, roll


class CallTimer:
    """CUDA-event pairs around C-ABI calls on the current stream."""

    def __init__(self):
        self.ev = {}

    def wrap(self, name, fn):
        import torch

        def inner(*a, **k):
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record()
            r = fn(*a, **k)
            e.record()
            self.ev.setdefault(name, []).append((s, e))
            return r
        return inner

    def mean_ms(self, name):
        xs = [s.elapsed_time(e) for s, e in self.ev.get(name, [])]
        return (sum(xs) / len(xs), len(xs)) if xs else (None, 0)


def max_over_ranks(values, device):
    """Element-wise maximum of a list of per-rank floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def replicas_throughput(world, units_per_step, steps, ms):
    """Whole-job units per second of `world` independent replicas that each did `steps` steps in `ms`
    milliseconds (the slowest rank's time)."""
    return world * units_per_step * steps / (ms * 1e-3)


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2509_16434_b200 import binding as ppo
    from paper_2509_16434_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    w = synth.WORKLOADS[args.workload]
    peaks = load_peaks()
    L, roll = make_learner(w, args.microbatch, device)

    timer = CallTimer()
    gather_name = "ppo_shuffle_gather_sequences" if w.n_lstm else "ppo_shuffle_gather_minibatch"
    names = ["ppo_compute_gae", gather_name, "ppo_encoder_fwd", "ppo_loss_fwd_bwd", "ppo_encoder_bwd", "ppo_adam_step"]
    originals = {n: getattr(ppo, n) for n in names}

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def one_step(seed):
        L.train(roll["last_value"], seed=seed)

    for i in range(args.warmup):
        one_step(i)
    barrier()
    for n in names:
        setattr(ppo, n, timer.wrap(n, originals[n]))
    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",")
    sampler = ClockSampler(vis[local] if local < len(vis) and vis[local].strip().isdigit() else local)
    launches0 = ppo.ppo_launch_count()
    if rank == 0:
        sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.nvtx.range_push("timed")
    t0.record()
    for i in range(args.steps):
        one_step(100 + i)
    t1.record()
    barrier()
    torch.cuda.nvtx.range_pop()
    clocks = sampler.stop() if rank == 0 else None
    for n in names:
        setattr(ppo, n, originals[n])
    ms = t0.elapsed_time(t1)
    status = ppo.ppo_poll_status()
    if status != 0:
        raise RuntimeError(f"device status {status} ({ppo.ppo_status_string(status)})")
    launches = ppo.ppo_launch_count() - launches0
    loss = L.loss.cpu().numpy().tolist()

    # ---- end to end: every step's rollout arrives from pinned host memory through ppo_buffer_write_step and the loss
    # scalars are read back.  Two device buffers alternate: the copies of the next rollout run on a second stream
    # while the learner trains on the current one (the simulator side collects while the learner trains), and a step
    # only starts once its own rollout has landed.
    host = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True) for k, v in roll.items()
            if k in ("depth", "proprio", "action", "logp", "value", "reward", "done", "last_value")}
    for k in host:
        host[k].copy_(roll[k])
    del roll["depth"]
    torch.cuda.empty_cache()
    stage = [{k: torch.empty_like(host[k][0], device=device) for k in host if k != "last_value"} for _ in range(2)]
    lastv = [torch.empty_like(roll["last_value"]) for _ in range(2)]
    h2d = sum(v.numel() * v.element_size() for v in host.values())
    loss_host = torch.empty(5, dtype=torch.float32, pin_memory=True)
    bufs = [L.buffer, ppo.Buffer(L.bdesc, device)]
    copy_stream = torch.cuda.Stream(device=device)
    landed = [torch.cuda.Event(), torch.cuda.Event()]
    trained = [torch.cuda.Event(), torch.cuda.Event()]
    main = torch.cuda.current_stream()

    def upload(i):
        """Rollout of step i -> buffer i % 2, on the copy stream, once that buffer's previous training is done."""
        b = i % 2
        copy_stream.wait_event(trained[b])
        with torch.cuda.stream(copy_stream):
            for t in range(w.T):
                st = stage[t % 2]
                for k in st:
                    st[k].copy_(host[k][t], non_blocking=True)
                ppo.ppo_buffer_write_step(bufs[b], t, st["depth"], st["proprio"], st["action"], st["logp"],
                                          st["value"], st["reward"], st["done"], stream=copy_stream)
            lastv[b].copy_(host["last_value"], non_blocking=True)
            landed[b].record(copy_stream)

    def e2e_run(n, seed0):
        for b in range(2):
            trained[b].record(main)
        upload(0)
        for i in range(n):
            b = i % 2
            if i + 1 < n:
                upload(i + 1)
            main.wait_event(landed[b])
            L.buffer = bufs[b]
            L.train(lastv[b], seed=seed0 + i)
            trained[b].record(main)
            loss_host.copy_(L.loss, non_blocking=True)
            main.synchronize()

    e2e_steps = max(1, min(args.steps, 5))
    e2e_run(2, 7)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    e2e_run(e2e_steps, 200)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    L.buffer = bufs[0]
    del bufs[1]

    ms, e2e_ms = max_over_ranks([ms, e2e_ms], device)
    env_steps = w.M * w.epochs
    value = replicas_throughput(world, env_steps, args.steps, ms)
    e2e_value = replicas_throughput(world, env_steps, e2e_steps, e2e_ms)

    if rank == 0:
        # roofline of the dominant calls: encoder forward+backward (tensor-bound), beside the HBM-bound ones
        rows = L.microbatch
        fwd_ms, n_fwd = timer.mean_ms("ppo_encoder_fwd")
        bwd_ms, _ = timer.mean_ms("ppo_encoder_bwd")
        gat_ms, _ = timer.mean_ms(gather_name)
        gae_ms, _ = timer.mean_ms("ppo_compute_gae")
        # the single-launch variant of GAE + moments + normalisation (scan, grid barrier, normalise), outside the step
        gae1 = []
        for i in range(8):
            s_, e_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s_.record()
            ppo.ppo_compute_gae(L.buffer, lastv[0], w.gamma, w.lam, 2, L.stats)
            e_.record()
            torch.cuda.synchronize()
            if i >= 3:
                gae1.append(s_.elapsed_time(e_))
        gae1_ms = float(np.median(gae1))
        adam_ms, _ = timer.mean_ms("ppo_adam_step")
        # a trailing micro-batch may be smaller; use the true mean rows per call
        calls_per_mb = -(-w.B // rows)
        mean_rows = w.B / calls_per_mb
        enc_flops = (fwd_flops_per_sample(w) + bwd_flops_per_sample(w)) * mean_rows
        enc_tf = enc_flops / ((fwd_ms + bwd_ms) * 1e-3) / 1e12
        peak_tf = peaks["bf16_tflops_sustained"]
        gather_gbs = 2 * (rows if w.n_lstm else w.B) * record_bytes(w) / (gat_ms * 1e-3) / 1e9
        gae_gbs = (17 + 8) * w.M / (gae_ms * 1e-3) / 1e9
        adam_gbs = 30 * L.model.arena / (adam_ms * 1e-3) / 1e9
        # DRAM bytes of the encoder's GEMM and conv1 kernels per sample row (dram__bytes_read + write summed over the 18
        # launches of one forward + backward, ncu capture of the cfg2 network at 512 rows: profiles/ncu_main_kernels_cfg2_prof.md);
        # traffic grows in proportion to the rows.  Valid for the cfg2/cfg3 network only, and only while those kernels are unchanged.
        per_row, capture = NCU_DRAM_BYTES_PER_ROW.get(w.name, (None, "no ncu capture of the current kernels at this workload"))
        traffic = per_row * mean_rows if per_row else None
        roofline = {"bound": "tensor",
                    "kernel": "ppo_encoder_fwd + ppo_encoder_bwd: tma_kmajor_kernel / tma_wgrad_kernel (tcgen05 implicit GEMMs) "
                              "+ conv1 kernels; flops, time and traffic per call pair",
                    "achieved": round(enc_tf, 2), "peak": peak_tf, "unit": "TFLOP/s",
                    "frac": round(enc_tf / peak_tf, 4), "traffic": traffic, "traffic_source": capture,
                    "peak_source": peaks["source"] + " (sustained bf16)",
                    "ms_per_call": {"fwd": round(fwd_ms, 4), "bwd": round(bwd_ms, 4), "rows": mean_rows}}
        others = {
            "gather": {"bound": "hbm", "achieved": round(gather_gbs, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                       "frac": round(gather_gbs / peaks["hbm_gbs"], 4), "ms": round(gat_ms, 4)},
            "gae_norm": {"bound": "hbm", "achieved": round(gae_gbs, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": round(gae_gbs / peaks["hbm_gbs"], 4), "ms": round(gae_ms, 4),
                         "note": "working set fits L2; launch-latency bound at this size",
                         "single_cooperative_launch_ms": round(gae1_ms, 4)},
            "adam": {"bound": "hbm", "achieved": round(adam_gbs, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": round(adam_gbs / peaks["hbm_gbs"], 4), "ms": round(adam_ms, 4),
                     "note": "working set fits L2; launch-latency bound at this size"},
        }
        others["supplementary_scaled_inputs"] = hbm_resident_rows(peaks)
        rollout = None if w.n_lstm else time_rollout_inference(L, host, w)
        cpu = cpu_baseline(w, host, L) if world == 1 and not args.no_cpu_baseline else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps,
            "ms_per_step_x_sm_ghz": (ms / args.steps * clocks["sm_mhz"] / 1e3) if clocks and clocks.get("sm_mhz") else None,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{w.name}: {w.N} envs x T={w.T}, depth 1x{w.H}x{w.W} fp16, conv "
                                   f"{'-'.join(map(str, w.conv_c))}, "
                                   + (f"{w.n_lstm} x LSTM({w.lstm_h}), " if w.n_lstm else "") +
                                   f"fc {'-'.join(map(str, w.fc))}, "
                                   f"{w.epochs} epoch(s) x {w.minibatches} minibatches",
                       "env_steps_per_step": env_steps, "minibatch": w.B, "microbatch": L.microbatch,
                       "l2_policy": "inputs_larger_than_l2 (buffer %.0f MB, minibatch activations %.0f MB)" % (
                           w.M * record_bytes(w) / 1e6, L.model.workspace.numel() / 1e6),
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 20,
                    "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                    "pipeline": "two device buffers; the next rollout's copies overlap the current step's training"},
            "gpu_launches": launches, "clocks": clocks, "roofline": roofline, "roofline_other_kernels": others,
            "cpu_baseline": cpu, "loss_last_minibatch": loss, "rollout_inference": rollout,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def time_rollout_inference(L, host, w, calls=8):
    """The step before the path (Algorithm 2, actions <- pi(obs), D <- D U {...}): the observation of one time step is
    written into its slab row, the encoder runs on it there and action, log-prob and value land in the same row
    (ppo_buffer_write_obs + ppo_policy_act over all N envs), outside the timed region of the headline metric."""
    import torch
    dev = L.device
    depth = host["depth"][0].to(dev)
    proprio = host["proprio"][0].to(dev)
    eps = torch.randn((w.N, w.A), device=dev)
    for t in range(min(2, w.T)):
        L.act_into_buffer(t, depth, proprio, eps)
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    s.record()
    for i in range(calls):
        L.act_into_buffer(i % w.T, depth, proprio, eps)
    e.record()
    torch.cuda.synchronize()
    ms = s.elapsed_time(e) / calls
    return {"value": w.N / (ms * 1e-3), "unit": "env-steps acted/s", "ms_per_call": round(ms, 4), "rows": w.N,
            "note": "ppo_buffer_write_obs + ppo_policy_act over all envs of one time step; not part of `value`"}


def hbm_resident_rows(peaks, warmup=3, steps=10):
    """Supplementary, HBM-resident inputs (NOT configs): the GAE and Adam kernels on working sets far larger than L2,
    to show their asymptotic bandwidth; at config sizes both finish inside a launch latency."""
    import torch
    from paper_2509_16434_b200 import binding as ppo
    extra = []
    T, N = 128, 524288
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    reward = torch.randn((T, N), generator=g, device="cuda")
    value = torch.randn((T, N), generator=g, device="cuda")
    done = (torch.rand((T, N), generator=g, device="cuda") < 0.01).to(torch.uint8)
    lastv = torch.randn(N, generator=g, device="cuda")
    adv, ret = torch.empty_like(reward), torch.empty_like(reward)
    ms = []
    for it in range(warmup + steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ppo.ppo_gae_static(reward, value, done, lastv, 0.99, 0.95, True, adv, ret)
        e1.record()
        torch.cuda.synchronize()
        if it >= warmup:
            ms.append(e0.elapsed_time(e1))
    t = float(np.median(ms))
    gbs = (17 + 8) * T * N / (t * 1e-3) / 1e9
    extra.append({"kernel": "gae_scan + adv_normalize", "input": f"{N} envs x T={T} ({(17 + 8) * T * N / 1e9:.2f} GB moved)",
                  "ms": round(t, 3), "GBs": round(gbs, 1), "frac_of_measured_hbm": round(gbs / peaks["hbm_gbs"], 4)})
    del reward, value, done, adv, ret
    md = ppo.model_desc(16, 16, (8,), (3,), (16384, 16384), 32, 12)
    model = ppo.Model(md, 1)
    model.grad.normal_(generator=g)
    ms = []
    for it in range(warmup + steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ppo.ppo_adam_step(model, 3e-4, 0.9, 0.999, 1e-8, it + 1)
        e1.record()
        torch.cuda.synchronize()
        if it >= warmup:
            ms.append(e0.elapsed_time(e1))
    t = float(np.median(ms))
    gbs = 30 * model.arena / (t * 1e-3) / 1e9
    extra.append({"kernel": "adam_kernel", "input": f"{model.arena} parameters ({30 * model.arena / 1e9:.2f} GB moved)",
                  "ms": round(t, 3), "GBs": round(gbs, 1), "frac_of_measured_hbm": round(gbs / peaks["hbm_gbs"], 4)})
    del model
    torch.cuda.empty_cache()
    return extra


# ---------------------------------------------------------------- CPU baseline ----

def sample_rows(w, n_samples):
    """Buffer rows (t * N + n) of the bounded sample, in the order the oracle trains on them: the first n_samples of the
    sample permutation, or, for a recurrent policy, the first n_samples / T envs of the env permutation, time-major."""
    from oracle import oracle as orc
    if not w.n_lstm:
        return orc.perm(w.seed, 0, w.M, 0, n_samples).astype(np.int64)
    envs = orc.perm(w.seed, 0, w.N, 0, n_samples // w.T).astype(np.int64)
    return (np.arange(w.T, dtype=np.int64)[:, None] * w.N + envs[None, :]).reshape(-1)


def oracle_sample_step(w, fields, theta, n_samples):
    """The oracle's learner step on a bounded sample: GAE + normalisation at full size, then one minibatch of
    n_samples rows (permutation, gather, forward, loss, backward, Adam).  Returns seconds and samples trained."""
    from oracle import oracle as orc
    md = orc.ModelDesc(w.H, w.W, tuple(w.conv_c), tuple(w.conv_k), tuple(w.fc), w.P, w.A, norm=w.norm, embed=w.embed,
                       n_lstm=w.n_lstm, lstm_h=w.lstm_h)
    t0 = time.perf_counter()
    adv, ret = orc.gae(fields["reward"], fields["value"], fields["done"], fields["last_value"], w.gamma, w.lam)
    adv, _, _ = orc.adv_normalize(adv)
    t_gae = time.perf_counter() - t0
    t0 = time.perf_counter()
    idx = sample_rows(w, n_samples)
    tt, nn = np.divmod(idx, w.N)
    depth = fields["depth_rows"]            # the sampled rows' frames, gathered on the device side of the bench
    g = {"proprio": fields["proprio"][tt, nn], "action": fields["action"][tt, nn], "logp": fields["logp"][tt, nn],
         "adv": adv[tt, nn], "ret": ret[tt, nn]}
    if w.n_lstm:
        ne = n_samples // w.T
        zero = np.zeros((w.n_lstm, ne, w.lstm_h))
        _, out, grad, _, _ = orc.total_loss_and_grad_seq(
            md, theta, depth.reshape(w.T, ne, w.H, w.W), g["proprio"].reshape(w.T, ne, w.P),
            fields["done"][tt, nn].reshape(w.T, ne), zero, zero, g["action"], g["logp"], g["adv"], g["ret"], w.clip, 0.5,
            0.01, act_bf16=True)
    else:
        _, out, grad, _, _ = orc.total_loss_and_grad(md, theta, depth, g["proprio"], g["action"], g["logp"], g["adv"],
                                                     g["ret"], w.clip, 0.5, 0.01, act_bf16=True)
    th = np.asarray(theta, np.float64).copy()
    orc.adam(th, np.zeros_like(th), np.zeros_like(th), grad, 3e-4, 0.9, 0.999, 1e-8, 1)
    t_mb = time.perf_counter() - t0
    return t_gae, t_mb, out


def cpu_baseline(w, host, L, n_samples=None):
    """Times the oracle, as it stands, on this machine's host cores over a bounded sample of the same workload."""
    from oracle import oracle as orc
    import torch
    # about 10-30 s of oracle work on a 16-core host: ~0.4 / 7 / 35 ms per row at the three frame sizes
    n_samples = n_samples or min(w.B, 4096 if w.H * w.W <= 120 * 160 else 768)
    if w.n_lstm:  # whole env sequences; the recurrent layers cost the oracle several times the CNN's time per row
        n_samples = max(1, min(n_samples, 1024) // w.T) * w.T
    idx = sample_rows(w, n_samples)
    flat = host["depth"].view(w.M, w.H, w.W)   # the rollout as it sits in pinned host memory
    fields = {k: host[k].numpy() for k in ("proprio", "action", "logp", "value", "reward", "done", "last_value")}
    fields["depth_rows"] = flat[torch.as_tensor(idx)].numpy()
    theta = L.model.master.cpu().numpy()
    t_gae, t_mb, _ = oracle_sample_step(w, fields, theta, n_samples)
    # whole step = GAE once + M*E sample-passes at the measured per-sample minibatch cost
    per_step = t_gae + t_mb / n_samples * w.M * w.epochs
    return {"value": w.M * w.epochs / per_step, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"GAE+normalisation at full size ({w.M} env-steps, {t_gae:.3f} s) + one minibatch of "
                      f"{n_samples} rows gather/fwd/loss/bwd/Adam ({t_mb:.2f} s), extrapolated linearly to "
                      f"{w.M * w.epochs} sample-passes"}


def run_reference(args):
    """The reference arm of this build is the CPU oracle: timed as it stands on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as orc
    from paper_2509_16434_b200 import synth
    w = synth.WORKLOADS[args.workload]
    # every step is a bounded sample; the default 3 + 5 steps stay within a few minutes of host time
    n_samples = min(w.B, 1024 if w.H * w.W <= 64 * 64 else 512 if w.H * w.W <= 120 * 160 else 96)
    if w.n_lstm:
        n_samples = max(1, n_samples // w.T) * w.T  # whole env sequences
    # a host-generated slice of the workload: all small fields at full size, frames only for the sampled rows
    small = w.scaled(w.N, H=2, W=2)
    roll = synth.rollout_numpy(small, w.seed)
    g = np.random.Generator(np.random.Philox(key=[w.seed, 1234]))
    depth = g.uniform(0.1, 2.0, (n_samples, w.H, w.W)).astype(np.float16)
    depth[g.random(depth.shape) < 0.1] = 0
    md = orc.ModelDesc(w.H, w.W, tuple(w.conv_c), tuple(w.conv_k), tuple(w.fc), w.P, w.A, norm=w.norm, embed=w.embed,
                       n_lstm=w.n_lstm, lstm_h=w.lstm_h)
    lay = orc.param_layout(md)
    theta = synth.init_params(lay.total, lay.offsets, lay.shapes, w.seed, ones=synth.param_shapes(w)[1])
    fields = {k: roll[k] for k in ("proprio", "value", "reward", "done", "last_value")}
    fields["action"] = roll["eps"]
    fields["logp"] = (-0.5 * (roll["eps"].astype(np.float64) ** 2).sum(-1) - 0.5 * w.A * np.log(2 * np.pi)
                      + roll["logp_jitter"]).astype(np.float32)
    fields["depth_rows"] = depth
    times = []
    for i in range(args.warmup + args.steps):
        t_gae, t_mb, _ = oracle_sample_step(w, fields, theta, n_samples)
        if i >= args.warmup:
            times.append(t_gae + t_mb / n_samples * w.M * w.epochs)
    per_step = float(np.mean(times))
    value = w.M * w.epochs / per_step
    sample = (f"per step: GAE+normalisation at full size + one minibatch of {n_samples} rows "
              f"(gather/fwd/loss/bwd/Adam), extrapolated linearly to {w.M * w.epochs} sample-passes")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(args.gpus),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name}: {w.N} envs x T={w.T}, depth 1x{w.H}x{w.W}", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_stress(args):
    """Bandwidth stress (GAE + advantage normalisation + one epoch of minibatch gathers only, T = 32) at
    1024 / 4096 / 16384 envs: achieved GB/s of the gather and of GAE against the measured HBM copy peak."""
    import torch
    from paper_2509_16434_b200 import binding as ppo
    from paper_2509_16434_b200 import synth
    torch.cuda.set_device(0)
    peaks = load_peaks()
    rows = []
    for name in ("cfg5_1k", "cfg5_4k", "cfg5_16k"):
        w = synth.WORKLOADS[name]
        desc = ppo.buffer_desc(w.N, w.T, w.H, w.W, w.P, w.A)
        buf = ppo.Buffer(desc)
        g = torch.Generator(device="cuda")
        g.manual_seed(w.seed)
        # fill the slabs in place (the frames of a 20 GB buffer are generated slab by slab)
        depth = buf.field(ppo.FIELD_DEPTH)
        for t in range(w.T):
            u = torch.rand(depth[t].shape, generator=g, device="cuda")
            z = torch.rand(depth[t].shape, generator=g, device="cuda") < 0.10
            depth[t].copy_((0.1 + 1.9 * u).to(torch.float16))
            depth[t][z] = 0
            del u, z
        for f in (ppo.FIELD_PROPRIO, ppo.FIELD_ACTION, ppo.FIELD_LOGP, ppo.FIELD_VALUE, ppo.FIELD_REWARD):
            buf.field(f).copy_(torch.randn(buf.field(f).shape, generator=g, device="cuda"))
        buf.field(ppo.FIELD_DONE).copy_((torch.rand((w.T, w.N), generator=g, device="cuda") < w.done_rate).to(torch.uint8))
        last_value = torch.randn(w.N, generator=g, device="cuda")
        mb = ppo.MinibatchArrays(desc, w.B, with_index=False)
        ev = lambda: torch.cuda.Event(enable_timing=True)
        gae_ms, gat_ms = [], []
        for it in range(args.warmup + args.steps):
            e0, e1, e2 = ev(), ev(), ev()
            e0.record()
            ppo.ppo_compute_gae(buf, last_value, w.gamma, w.lam, True, None)
            e1.record()
            for k in range(w.minibatches):
                ppo.ppo_shuffle_gather_minibatch(buf, it, 0, k, w.minibatches, mb)
            e2.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                gae_ms.append(e0.elapsed_time(e1))
                gat_ms.append(e1.elapsed_time(e2))
        gae, gat = float(np.median(gae_ms)), float(np.median(gat_ms))
        gather_gbs = 2 * w.M * record_bytes(w) / (gat * 1e-3) / 1e9
        gae_gbs = (17 + 8) * w.M / (gae * 1e-3) / 1e9
        rows.append({"workload": name, "envs": w.N, "T": w.T, "buffer_GB": round(w.M * record_bytes(w) / 1e9, 2),
                     "gather_ms_per_epoch": round(gat, 3), "gather_GBs": round(gather_gbs, 1),
                     "gather_frac_of_measured_hbm": round(gather_gbs / peaks["hbm_gbs"], 4),
                     "gae_norm_ms": round(gae, 4), "gae_norm_GBs": round(gae_gbs, 1),
                     "gae_norm_frac_of_measured_hbm": round(gae_gbs / peaks["hbm_gbs"], 4)})
        assert ppo.ppo_poll_status() == 0
        del buf, mb, depth
        torch.cuda.empty_cache()
    extra = hbm_resident_rows(peaks, args.warmup, args.steps)
    print(json.dumps({"metric": "buffer_path_bandwidth", "unit": "GB/s", "peak_hbm_gbs": peaks["hbm_gbs"],
                      "peak_source": peaks["source"], "rows": rows, "supplementary_scaled_inputs": extra}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--microbatch", type=int, default=4096)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--stress", action="store_true", help="bandwidth stress of the buffer path (GAE + gathers, T = 32)")
    args = ap.parse_args()
    if args.stress:
        run_stress(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
