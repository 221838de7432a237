#!/usr/bin/env python
"""Throughput of the sample production/consumption path on synthetic workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl ours|reference]

One pass of the whole path is: the workload's producer:consumer ratio of actor steps (one tj_actor_step call), then
one learner step (tj_replay_sample + tj_td_error, or tj_segment_acquire + tj_gae for the on-policy workload), then
one tj_publish_weights (a new version).  One "step" repeats that pass `patterns_per_step` times (config key), chosen
per workload so that 20 steps keep the GPU busy for about a second: the clock sampler then sees the load, and the
roofline fraction is taken against the sustained peak.
`value` is env-steps per second with everything resident in HBM; `e2e` is the same loop with the parameter
blob coming from pinned host memory and the TD errors and loss read back to the host every pass.
N > 1 runs N independent replicas (the path does not shard), one process per GPU: under a launcher that sets
WORLD_SIZE this process is one rank; without one, `--gpus N` starts the N ranks itself.
`--sweep` adds consumed samples per second for each staleness bound the workload's configuration names.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2502_20190_b200 import synth  # noqa: E402

# dram__bytes (read + write) per env-step of the fused tensor-core actor launch, from one ncu capture of the kernel as it
# stands (a smaller number of envs, scaled: traffic grows with the number of envs).  None once the kernel has changed
# since the counters were taken.
NCU_DRAM_BYTES_PER_ENV_STEP = {"cfg5": 1990.0}   # 226.3 MB per launch of 113,664 envs
L2_FLUSH_BYTES = 256 << 20
# passes of the path per bench step: about 50 ms of GPU time per step
PATTERNS_PER_STEP = {"cfg1": 512, "cfg2": 256, "cfg3": 128, "cfg4": 8, "cfg5": 64}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                    sm_max_mhz=d.get("sm_max_mhz", 1965.0), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, sm_max_mhz=1965.0, source="fallback")


def mlp_macs(w):
    D, H, A = w["obs_dim"], w["hidden"], w["n_actions"] + (1 if w["policy_kind"] == 1 else 0)
    return D * H + H * H + H * A


def actor_algorithmic(w):
    """(flops, bytes) one env-step must spend: the policy MLP (+ the env's mat-vec) and state read+write,
    counters, one record written."""
    D = w["obs_dim"]
    S_d = D if w["env_kind"] == synth.ENV_LINGAUSS else 4
    flops = 2 * mlp_macs(w) + (2 * D * D if w["env_kind"] == synth.ENV_LINGAUSS else 0)
    if w["replay_capacity"]:
        rec = (2 * D + 4) * 4
    else:
        rec = D * 4 + 4 + 4 + 1 + 4 + 4
    return flops, 2 * S_d * 4 + 8 + rec


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def max_over_ranks(values, device):
    """Element-wise maximum of per-rank timings over all ranks (the job runs as long as its slowest replica)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def min_over_ranks(values, device):
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MIN)
    return [float(x) for x in t.tolist()]


def aggregate_throughput(units_per_replica, world, max_ms):
    """Whole-job rate of `world` independent replicas that each processed units_per_replica in max_ms."""
    return units_per_replica * world / (max_ms * 1e-3)


# --------------------------------------------------------------------------------------------- our arm
class Runner:
    """Drives one context through the workload's call pattern."""

    def __init__(self, name, torch, binding, device_index, n_envs=0, with_update=False, two_stream=False, tensor_fp32=None):
        self.torch, self.name = torch, name
        self.w = dict(synth.WORKLOADS[name])
        if tensor_fp32 is None:
            # default: the FP32 workloads whose hidden x hidden layer is a dense contraction (hidden >= 256: cfg3, cfg4) run it
            # on the tensor cores at FP32 accuracy; --fp32-fma selects the bit-reproducible FMA kernel instead
            tensor_fp32 = (self.w["weight_dtype"] == synth.W_FP32 and self.w["env_kind"] != synth.ENV_LINGAUSS
                           and self.w["hidden"] in (256,))
        if tensor_fp32:
            # FP32 weights, the actor's hidden x hidden layer as split-operand tensor-core products (1e-5 of the FP32 path)
            if self.w["weight_dtype"] != synth.W_FP32 or self.w["env_kind"] == synth.ENV_LINGAUSS or self.w["hidden"] % 64:
                raise SystemExit("--tensor-fp32 applies to the FP32 CartPole / Acrobot workloads with hidden 64..256")
            self.w["weight_dtype"] = synth.W_FP32_TC
        if n_envs:
            if self.w["replay_capacity"]:
                self.w["replay_capacity"] = self.w["replay_capacity"] // self.w["n_envs"] * n_envs
            self.w["n_envs"] = n_envs
        self.f = synth.config_fields(self.w, device=device_index)
        self.ctx = binding.Context(**self.f)
        self.on_policy = self.w["replay_capacity"] == 0
        self.actor_steps = self.w["rollout_len"] if self.on_policy else self.w["actor_per_learner"]
        vh = self.w["policy_kind"] == 1
        D, H, A = self.w["obs_dim"], self.w["hidden"], self.w["n_actions"]
        # a small pool of parameter versions, on the device and in pinned host memory
        self.n_pool = 8
        blobs = [synth.policy_blob(self.f["seed"], v + 1, D, H, A, vh) for v in range(self.n_pool)]
        self.dev_blobs = [torch.from_numpy(b).cuda() for b in blobs]
        self.host_blobs = [torch.from_numpy(b).pin_memory() for b in blobs]
        self.version = 0
        self.learner_ok = 0
        # --with-update: the learner also takes a gradient step (tj_sgd_step) and the published parameters are the ones it
        # trains, instead of the pre-drawn pool (replay workloads only; FP32 master parameters in BF16 workloads too)
        self.with_update = bool(with_update) and self.w["replay_capacity"] > 0
        if self.with_update:
            self.theta = self.dev_blobs[0].clone()
            self.theta_target = self.dev_blobs[0].clone()
            self.lr = 1e-3
        if not self.on_policy:
            self.batch = self.ctx.alloc_batch()
            B = self.w["minibatch"]
            self.out = dict(td=torch.empty(B, dtype=torch.float32, device="cuda"),
                            huber=torch.empty(B, dtype=torch.float32, device="cuda"),
                            loss=torch.empty(1, dtype=torch.float32, device="cuda"))
            self.host_td = torch.empty(B, dtype=torch.float32).pin_memory()
            self.host_loss = torch.empty(1, dtype=torch.float32).pin_memory()
        else:
            T, N = self.w["rollout_len"], self.w["n_envs"]
            self.adv = torch.empty((T, N), dtype=torch.float32, device="cuda")
            self.ret = torch.empty((T, N), dtype=torch.float32, device="cuda")
            self.host_adv_mean = torch.empty(1, dtype=torch.float32).pin_memory()
        self.publish(False)
        # --two-stream: the learner's calls on a second CUDA stream; a pass then runs the learner on what was produced so far,
        # the actor's next block beside it, and the publish last (replay workloads)
        self.two_stream = bool(two_stream) and not self.on_policy
        if self.two_stream:
            self.ctx.use_learner_stream(True)
            self.lstream = self.ctx.learner_stream
            self.actor()

    def publish(self, from_host):
        if self.with_update:
            self.ctx.publish_weights(self.theta)
            self.version += 1
            if self.version % 1000 == 0:
                if getattr(self, "two_stream", False):
                    with self.torch.cuda.stream(self.lstream):
                        self.theta_target.copy_(self.theta)
                else:
                    self.theta_target.copy_(self.theta)
            return
        blob = (self.host_blobs if from_host else self.dev_blobs)[self.version % self.n_pool]
        if from_host:
            from paper_2502_20190_b200 import binding as b
            st, _ = b.tj_publish_weights(self.ctx.h, blob.data_ptr(), blob.numel() * 4, 0)
            assert st == 0, b.tj_last_error(self.ctx.h)
        else:
            self.ctx.publish_weights(blob)
        self.version += 1

    def actor(self):
        self.ctx.actor_step(self.actor_steps)

    def learner(self):
        if self.on_policy:
            st, seg = self.ctx.segment_acquire(allow=(0, -7))
            if st == 0:
                self.ctx.gae(seg["rew"], seg["val"], seg["done"], self.w["gamma"], self.w["gae_lambda"], self.adv, self.ret)
                self.learner_ok += 1
        else:
            st, _ = self.ctx.replay_sample(batch=self.batch, allow=(0, -6, -7))
            if st == 0:
                self.ctx.td_error(self.batch, self.out)
                if self.with_update:
                    self.ctx.sgd_step(self.batch, self.lr, self.theta, self.theta_target)
                self.learner_ok += 1

    def one_pass(self, e2e=False):
        torch = self.torch
        if self.two_stream:
            self.learner()
            self.actor()
            self.publish(e2e)
            if e2e:
                with torch.cuda.stream(self.lstream):
                    self.host_td.copy_(self.out["td"], non_blocking=True)
                    self.host_loss.copy_(self.out["loss"], non_blocking=True)
                self.lstream.synchronize()
                torch.cuda.current_stream().synchronize()
            return
        self.actor()
        self.learner()
        self.publish(e2e)
        if e2e:
            if self.on_policy:
                self.host_adv_mean.copy_(self.adv[0, :1], non_blocking=True)
            else:
                self.host_td.copy_(self.out["td"], non_blocking=True)
                self.host_loss.copy_(self.out["loss"], non_blocking=True)
            torch.cuda.current_stream().synchronize()

    def step(self, patterns, events=None, e2e=False):
        if events:
            events[0].record()
        for _ in range(patterns):
            self.one_pass(e2e)
        if self.two_stream:      # the step ends when both streams have finished it
            self.torch.cuda.current_stream().wait_event(self.lstream.record_event())
        if events:
            events[1].record()

    def e2e_bytes(self):
        h2d = 0 if self.with_update else self.host_blobs[0].numel() * 4
        d2h = 4 if self.on_policy else (self.w["minibatch"] + 1) * 4
        return h2d, d2h


def class_bytes(w, name, on_policy):
    """Algorithmic HBM bytes one launch group of a memory-bound kernel class must move (None: not memory-bound)."""
    D, A = w["obs_dim"], w["n_actions"]
    if name == "sample_gather":       # sampled records read, the same bytes written as dense arrays, indices
        return 2 * w["minibatch"] * (2 * D + 4) * 4 + w["minibatch"] * 4
    if name == "td" and w["weight_dtype"] == synth.W_BF16:   # elementwise pass after the tensor-core forwards
        return w["minibatch"] * (2 * A * 4 + 3 * 4 + 2 * 4)
    if name == "gae":                 # rew, val, done read; adv, ret written
        return w["rollout_len"] * w["n_envs"] * 17
    return None


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2502_20190_b200 import binding, build
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    binding.load_library()
    peaks = load_peaks()
    name = args.workload
    if args.tensor_fp32 and args.fp32_fma:
        raise SystemExit("--tensor-fp32 and --fp32-fma exclude each other")
    r = Runner(name, torch, binding, local, args.envs, args.with_update, args.two_stream,
               True if args.tensor_fp32 else (False if args.fp32_fma else None))
    w = r.w
    N = w["n_envs"]
    R = args.patterns or PATTERNS_PER_STEP[name]
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    ring_bytes = w["replay_capacity"] * (2 * w["obs_dim"] + 4) * 4
    need_flush = ring_bytes < 4 * (126 << 20)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        r.step(R)
    barrier()

    def timed_loop(K, e2e):
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(K)]
        launches0 = r.ctx.stats()["kernel_launches"]
        r.learner_ok = 0
        for i in range(K):
            if need_flush:
                flush.fill_(i & 0xFF)
            r.step(R, evs[i], e2e)
        torch.cuda.synchronize()
        tot = sum(e[0].elapsed_time(e[1]) for e in evs)
        return tot, r.ctx.stats()["kernel_launches"] - launches0, r.learner_ok

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    t_wall = time.time()
    tot_ms, launches, learner_ok = timed_loop(args.steps, False)
    barrier()
    wall = time.time() - t_wall
    clocks = sampler.stop() if rank == 0 else None
    e2e_ms, _, _ = timed_loop(args.steps, True)
    barrier()
    # the same K steps once more with the library's per-kernel CUDA events on: duration of each kernel class
    r.ctx.set_profiling(1)
    timed_loop(args.steps, False)
    prof = r.ctx.stats()
    prof_learner_steps = r.learner_ok
    r.ctx.set_profiling(0)
    barrier()
    fp32_peak = r.ctx.calibrate_fp32() if (w["weight_dtype"] == synth.W_FP32 or r.with_update) else None

    tot_ms, e2e_ms = max_over_ranks([tot_ms, e2e_ms], "cuda")
    learner_ok = int(min_over_ranks([learner_ok], "cuda")[0])
    K = args.steps
    env_steps = N * r.actor_steps * R * K * world
    assert abs(aggregate_throughput(N * r.actor_steps * R * K, world, tot_ms) - env_steps / (tot_ms * 1e-3)) < 1e-6 * env_steps
    consumed = (w["rollout_len"] * N if r.on_policy else w["minibatch"]) * learner_ok * world
    value = env_steps / (tot_ms * 1e-3)
    flops, nbytes = actor_algorithmic(w)
    names = ["actor_fused", "mlp_tensor", "env_select_insert", "sample_gather", "td", "publish", "gae", "sgd_update"]
    kms, kcnt = prof["kernel_ms"], prof["kernel_count"]
    total_kms = sum(kms) or 1.0
    kernels = {}
    for i, nm in enumerate(names):
        if not kcnt[i]:
            continue
        kernels[nm] = {"launches": kcnt[i], "ms": kms[i], "share": kms[i] / total_kms, "us_per_launch": 1e3 * kms[i] / kcnt[i]}
        cb = class_bytes(w, nm, r.on_policy)
        if cb:      # memory-bound kernels taken alone, against the measured copy bandwidth
            groups = kcnt[i] if nm != "td" else kcnt[i] // 2 or 1   # td: elementwise pass + loss reduction per learner step
            gbs = cb * groups / (kms[i] * 1e-3) / 1e9
            kernels[nm].update({"algorithmic_bytes_per_call": cb, "achieved_gbs": gbs, "hbm_frac_of_measured": gbs / peaks["hbm_gbs"]})
    dom = max(range(len(names)), key=lambda i: kms[i])
    mlp_flops = 2 * mlp_macs(w)
    timed_s = tot_ms * 1e-3
    sustained = timed_s >= 1.0
    tensor_peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    tensor_peak_name = ("cuBLAS bf16 sustained (timed region %.2f s >= 1 s)" if sustained else "cuBLAS bf16 burst (timed region %.2f s < 1 s)") % timed_s
    if dom == 0 and w["weight_dtype"] == synth.W_BF16:
        # fused tensor-core actor: one launch = one env step for all N envs; MLP flops only, actor launches only
        us = 1e3 * kms[0] / kcnt[0]
        achieved = mlp_flops * N / (us * 1e-6) / 1e12
        roof = {"kernel": "actor_tc_pipelined_kernel (fused tcgen05 actor step: MLP + selection + A s + env step + insert)",
                "bound": "tensor", "achieved": achieved, "peak": tensor_peak, "unit": "TFLOP/s",
                "peak_source": tensor_peak_name + ", of " + peaks["source"], "us_per_launch": us,
                "units_per_launch": N, "flop_per_unit": mlp_flops,
                "hbm_view": {"bytes_per_unit": nbytes, "achieved_gbs": nbytes * N / (us * 1e-6) / 1e9,
                             "frac_of_measured": nbytes * N / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}}
    elif dom == 0 and w["weight_dtype"] == synth.W_FP32_TC:
        # split-operand tensor-core actor: one launch = actor_steps env steps; algorithmic MLP flops (the hidden x hidden
        # layer costs three tensor-core products per algorithmic product, so the pipe does about 3x this work)
        us = 1e3 * kms[0] / kcnt[0]
        units = N * r.actor_steps
        achieved = mlp_flops * units / (us * 1e-6) / 1e12
        roof = {"kernel": "actor_split_tc_kernel (FP32 layer 1 + FP16-split tcgen05 hidden layer + head + selection + env step + insert)",
                "bound": "tensor", "achieved": achieved, "peak": tensor_peak, "unit": "TFLOP/s",
                "peak_source": tensor_peak_name + ", of " + peaks["source"] + "; fp16 peak = bf16 peak", "us_per_launch": us,
                "units_per_launch": units, "flop_per_unit": mlp_flops, "tensor_products_per_algorithmic_product": 3,
                "hbm_view": {"bytes_per_unit": nbytes, "achieved_gbs": nbytes * units / (us * 1e-6) / 1e9,
                             "frac_of_measured": nbytes * units / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}}
    elif dom == 0:
        # fused FP32 actor kernel: one launch = actor_steps env steps for all N envs
        us = 1e3 * kms[0] / kcnt[0]
        units = N * r.actor_steps
        achieved = flops * units / (us * 1e-6) / 1e12
        roof = {"kernel": "actor_small_env_kernel (FP32 MLP + selection + env step + insert)", "bound": "alu",
                "achieved": achieved, "peak": fp32_peak, "unit": "TFLOP/s",
                "peak_source": "FP32 FMA loop on every SM, measured in this run (tj_calibrate_fp32)", "us_per_launch": us,
                "units_per_launch": units, "flop_per_unit": flops,
                "hbm_view": {"bytes_per_unit": nbytes, "achieved_gbs": nbytes * units / (us * 1e-6) / 1e9,
                             "frac_of_measured": nbytes * units / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}}
    elif dom == 1:
        us = 1e3 * kms[1] / kcnt[1]
        rows = N if kcnt[1] and not kcnt[0] and not r.on_policy and kcnt[2] else w["minibatch"]
        achieved = mlp_flops * rows / (us * 1e-6) / 1e12
        roof = {"kernel": "mlp_bf16_tc_kernel (tcgen05 MLP forward)", "bound": "tensor", "achieved": achieved,
                "peak": tensor_peak, "unit": "TFLOP/s", "peak_source": tensor_peak_name + ", of " + peaks["source"],
                "us_per_launch": us, "units_per_launch": rows, "flop_per_unit": mlp_flops}
    elif names[dom] == "sgd_update":
        # the learner's gradient step dominates: forward + backward = 6 flops per weight and row, against the FP32 FMA rate
        # (its weight-gradient products run as 3 x TF32 on the tensor cores, the rest on the FP32 pipes)
        ms_per_update = kms[dom] / max(prof_learner_steps, 1)       # learner steps of the profiled loop
        upd_flops = 6.0 * mlp_macs(w) * w["minibatch"]
        roof = {"kernel": "sgd_update (tj_sgd_step: forward, backward, Adam)", "bound": "alu",
                "achieved": upd_flops / (ms_per_update * 1e-3) / 1e12, "peak": fp32_peak, "unit": "TFLOP/s",
                "peak_source": "FP32 FMA loop on every SM, measured in this run (tj_calibrate_fp32)",
                "us_per_launch": 1e3 * kms[dom] / kcnt[dom], "ms_per_update": ms_per_update, "units_per_launch": w["minibatch"],
                "flop_per_unit": 6.0 * mlp_macs(w)}
    elif names[dom] == "td" and w["weight_dtype"] != synth.W_BF16:
        # FP32 TD kernel (online forward on obs, target forward on next_obs, then the elementwise error): two MLP passes per row
        us = 1e3 * kms[dom] / (kcnt[dom] // 2 or 1)                 # the class counts the loss reduction launch as well
        if fp32_peak is None:
            fp32_peak = r.ctx.calibrate_fp32()
        roof = {"kernel": "td_kernel (FP32 online + target forward, TD target, Huber) + loss reduction", "bound": "alu",
                "achieved": 2 * mlp_flops * w["minibatch"] / (us * 1e-6) / 1e12, "peak": fp32_peak, "unit": "TFLOP/s",
                "peak_source": "FP32 FMA loop on every SM, measured in this run (tj_calibrate_fp32)", "us_per_launch": us,
                "units_per_launch": w["minibatch"], "flop_per_unit": 2 * mlp_flops}
    else:
        # a memory-bound class dominates (GAE on the on-policy workload, gather on tiny ones)
        nm = names[dom]
        us = 1e3 * kms[dom] / kcnt[dom]
        cb = class_bytes(w, nm, r.on_policy) or 0
        roof = {"kernel": nm, "bound": "hbm", "achieved": cb / (us * 1e-6) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "peak_source": "copy bandwidth, of " + peaks["source"], "us_per_launch": us, "units_per_launch": 1,
                "bytes_per_unit": cb}
    roof["frac"] = roof["achieved"] / roof["peak"] if roof["peak"] else None
    per_env = NCU_DRAM_BYTES_PER_ENV_STEP.get(name) if (dom == 0 and w["weight_dtype"] == synth.W_BF16) else None
    roof["traffic"] = per_env * N if per_env else None
    roof["traffic_note"] = "bytes per fused actor launch (N env-steps), ncu capture at fewer envs scaled by N" if per_env else None
    if clocks and clocks.get("sm_mhz"):
        roof["sm_mhz_median_under_load"] = clocks["sm_mhz"]
    h2d, d2h = r.e2e_bytes()
    line = {
        "metric": "env-steps/s", "value": value, "unit": "env-steps/s", "n_gpus": world, "steps": K,
        "warmup": args.warmup, "ms_per_step": tot_ms / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w["weight_dtype"] == synth.W_BF16 else ("f32 (hidden layer: 3 x fp16 split products)" if w["weight_dtype"] == synth.W_FP32_TC else "f32"), "data": "synthetic",
        "config": {"workload": name, "n_envs": N, "patterns_per_step": R, "actor_steps_per_pattern": r.actor_steps,
                   "minibatch": w.get("minibatch"), "mlp": "%d-%d-%d-%d" % (w["obs_dim"], w["hidden"], w["hidden"], w["n_actions"]),
                   "replicas": world, "learner_update": r.with_update, "two_stream": r.two_stream, "weight_mode": {0: "fp32 fma", 1: "bf16 tensor", 2: "fp32 weights, split-operand tensor"}[w["weight_dtype"]],
                   "l2": "flushed between steps (256 MiB write outside the per-step event pairs)" if need_flush
                   else "ring larger than L2"},
        "consumed_samples_per_s": consumed / (tot_ms * 1e-3),
        "ms_per_pattern": tot_ms / K / R, "timed_region_s": timed_s, "wall_s": wall,
        "e2e": {"value": env_steps / (e2e_ms * 1e-3), "unit": "env-steps/s", "h2d_bytes_per_step": h2d * R,
                "d2h_bytes_per_step": d2h * R},
        "gpu_launches": launches,
        "roofline": roof,
        "kernels": kernels,
        "clocks": clocks,
    }
    if args.sweep and not r.on_policy:
        line["staleness_sweep"] = staleness_sweep(r, torch, w, R)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(name, budget_s=args.cpu_seconds)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def staleness_sweep(r, torch, w, R):
    """Consumed samples per second for each staleness bound the configuration names (Sec. 4.3.2, App. D.1): the same
    cadence (actor steps, one sample + TD error, publish), the sample call taking the bound; starved calls consume nothing."""
    out = []
    for bound in w.get("staleness_sweep", (w["staleness_bound"],)):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ok = starved = 0
        torch.cuda.synchronize()
        a.record()
        for _ in range(R * 4):
            r.actor()
            st, _ = r.ctx.replay_sample(bound, batch=r.batch, allow=(0, -6, -7))
            if st == 0:
                r.ctx.td_error(r.batch, r.out)
                ok += 1
            else:
                starved += 1
            r.publish(False)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b)
        out.append({"staleness_bound": bound, "consumed_samples_per_s": ok * w["minibatch"] / (ms * 1e-3),
                    "env_steps_per_s": R * 4 * r.actor_steps * w["n_envs"] / (ms * 1e-3), "learner_steps": ok, "starved_calls": starved})
    return out


# --------------------------------------------------------------------------------------------- oracle arm
def oracle_sample_shape(name, shards):
    """A bounded sample of the workload for the CPU oracle: a subsample of the envs (4,096 where the workload has more),
    cut into `shards` equal shards, each an oracle of its own with its own ring; the same call pattern."""
    w = synth.WORKLOADS[name]
    total = min(w["n_envs"], 4096)
    n_envs = max(total // shards, 1)
    over = dict(n_envs=n_envs)
    if w["replay_capacity"]:
        over["replay_capacity"] = n_envs * 64
        over["minibatch"] = max(w["minibatch"] * n_envs // w["n_envs"], 1)   # the workload's rows consumed per env-step
        over["warmup"] = over["minibatch"]
    return over


def oracle_step_fn(name, shards=1, shard=0):
    import oracle
    w = synth.WORKLOADS[name]
    over = oracle_sample_shape(name, shards)
    f = synth.config_fields(w, **over)
    f["seed"] = f["seed"] + shard
    o = oracle.Oracle(**f)
    vh = w["policy_kind"] == 1
    state = dict(v=0)
    on_policy = w["replay_capacity"] == 0
    a_steps = w["rollout_len"] if on_policy else w["actor_per_learner"]
    blobs = [synth.policy_blob(synth.SEED, v + 1, w["obs_dim"], w["hidden"], w["n_actions"], vh) for v in range(8)]

    def publish():
        state["v"] += 1
        o.publish(blobs[(state["v"] - 1) % 8])

    def step():
        o.actor_step(a_steps)
        consumed = 0
        if on_policy:
            st, seg = o.segment_acquire()
            if st == 0:
                oracle.gae(seg["rew"], seg["val"], seg["done"], w["gamma"], w["gae_lambda"])
                consumed = seg["T"] * seg["N"]
        else:
            st, _, rec = o.sample()
            if st == 0:
                o.td(rec)
                consumed = rec.shape[0]
        publish()
        return f["n_envs"] * a_steps, consumed

    publish()
    desc = "%d of %d envs per shard, %d actor steps + 1 learner step (minibatch %s) per pass" % (
        f["n_envs"], w["n_envs"], a_steps, f.get("minibatch"))
    return step, desc


class OracleShards:
    """The oracle as it stands on `threads` host threads, each stepping its own shard of the env subsample (the oracle's
    C routines run outside the interpreter lock)."""

    def __init__(self, name, threads):
        self.threads = threads
        fns = [oracle_step_fn(name, threads, i) for i in range(threads)]
        self.fns = [f for f, _ in fns]
        self.desc = fns[0][1]
        self.run(0.0)                          # one warm-up pass per shard (fills the ring past its warm-up size)

    def run(self, budget_s):
        """Step every shard for budget_s seconds; returns (env-steps/s, consumed samples/s, passes, seconds)."""
        import threading
        totals = [[0, 0, 0] for _ in range(self.threads)]
        t0 = time.time()
        deadline = t0 + budget_s

        def work(i):
            while True:
                e, c = self.fns[i]()
                totals[i][0] += e
                totals[i][1] += c
                totals[i][2] += 1
                if time.time() >= deadline:
                    break

        ths = [threading.Thread(target=work, args=(i,)) for i in range(self.threads)]
        for t in ths:
            t.start()
        for t in ths:
            t.join()
        dt = time.time() - t0
        return sum(t[0] for t in totals) / dt, sum(t[1] for t in totals) / dt, sum(t[2] for t in totals), dt


def host_threads():
    cores = os.cpu_count() or 1
    P = 1
    while P * 2 <= min(cores, 64):
        P *= 2
    return cores, P


def cpu_baseline(name, budget_s=16.0):
    cores, P = host_threads()
    one = OracleShards(name, 1)
    v1, c1, n1, dt1 = one.run(budget_s / 2)
    if P > 1:
        many = OracleShards(name, P)
        vp, cp, np_, dtp = many.run(budget_s / 2)
    else:
        many, (vp, cp, np_, dtp) = one, (v1, c1, n1, dt1)
    return {"value": vp, "unit": "env-steps/s", "cores": P, "kind": "oracle",
            "sample": "%d shards x (%s); %d passes in %.1f s on %d threads" % (P, many.desc, np_, dtp, P),
            "consumed_samples_per_s": cp,
            "single_thread": {"value": v1, "consumed_samples_per_s": c1, "cores": 1,
                              "sample": "%s; %d passes in %.1f s" % (one.desc, n1, dt1)},
            "host_cores": cores}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.workload
    w = synth.WORKLOADS[name]
    cores, P = host_threads()
    shards = OracleShards(name, P)
    # each step is a bounded sample: a fixed slice of host time on P threads, every thread stepping its own env shard
    per_step_s = max(0.5, min(3.0, 60.0 / max(args.steps + args.warmup, 1)))
    for _ in range(min(args.warmup, 3)):
        shards.run(0.2)
    env_steps = consumed = 0.0
    t0 = time.time()
    for _ in range(args.steps):
        v, c, _, dt_ = shards.run(per_step_s)
        env_steps += v * dt_
        consumed += c * dt_
    dt = time.time() - t0
    value = env_steps / dt
    sample = "%d shards x (%s) on %d threads, about %.1f s of stepping per bench step" % (P, shards.desc, P, per_step_s)
    line = {
        "impl": "reference", "metric": "env-steps/s", "value": value, "unit": "env-steps/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt * 1e3 / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": name, "n_envs": w["n_envs"], "sample": sample},
        "consumed_samples_per_s": consumed / dt,
        "cpu_baseline": {"value": value, "unit": "env-steps/s", "cores": P, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "env-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def spawn_replicas(args):
    """`--gpus N` without a launcher: start the N ranks (one process per GPU) and pass their output through."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg5", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--envs", type=int, default=0, help="profiling aid: run the workload with this many envs (ring scaled to the same number of steps)")
    ap.add_argument("--patterns", type=int, default=0, help="passes of the path per step (default: per workload, about 50 ms of GPU time)")
    ap.add_argument("--with-update", action="store_true", help="FP32 replay workloads: the learner step also runs tj_sgd_step and publishes the parameters it trains")
    ap.add_argument("--two-stream", action="store_true", help="replay workloads: learner calls on a second CUDA stream, passes software-pipelined (learner on the previous block beside the actor's next one)")
    ap.add_argument("--tensor-fp32", action="store_true", help="FP32 CartPole / Acrobot workloads: weight mode TJ_W_FP32_TC (hidden x hidden layer on the tensor cores as split-operand products, 1e-5 of the FP32 path)")
    ap.add_argument("--fp32-fma", action="store_true", help="FP32 workloads: weight mode TJ_W_FP32 (FMA kernel, one fixed rounding order) also where the tensor-core mode is the default (hidden 256)")
    ap.add_argument("--sweep", action="store_true", help="also report consumed samples/s for each staleness bound the workload names")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=16.0)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    world = os.environ.get("WORLD_SIZE")
    if args.impl == "ours" and args.gpus > 1:
        if world is None:
            raise SystemExit(spawn_replicas(args))
        if int(world) != args.gpus:
            raise SystemExit("bench.py: --gpus %d but the launcher started %s ranks" % (args.gpus, world))
    elif args.impl == "ours" and world is not None and int(world) != args.gpus:
        raise SystemExit("bench.py: --gpus %d but the launcher started %s ranks" % (args.gpus, world))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
