#!/usr/bin/env python
"""Throughput of the sample production/consumption path on synthetic workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl ours|reference]

One "step" is one pass of the whole path over one batch: the workload's producer:consumer ratio of actor
steps (one tj_actor_step call), then one learner step (tj_replay_sample + tj_td_error, or
tj_segment_acquire + tj_gae for the on-policy workload), then one tj_publish_weights (a new version).
`value` is env-steps per second with everything resident in HBM; `e2e` is the same loop with the parameter
blob coming from pinned host memory and the TD errors and loss read back to the host every step.
N > 1 runs N independent replicas (the path does not shard), one process per GPU.
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

SM_COUNT, FMA_LANES_PER_SM = 148, 128
# dram__bytes (read + write) per env-step of the pipelined tensor-core actor launch, from one ncu capture of the kernel as
# it stands (113,664 envs: 1.320 TB/s over 188.6 us = 249.0 MB per launch); traffic grows with the number of envs.  Set to
# None when the kernel changes.  See profiles/cfg5_pipelined_tensor_core_actor.md.
NCU_DRAM_BYTES_PER_ENV_STEP = {"cfg5": 2190.7}
L2_FLUSH_BYTES = 256 << 20


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

    def __init__(self, name, torch, binding, device_index, n_envs=0, with_update=False):
        self.torch, self.name = torch, name
        self.w = dict(synth.WORKLOADS[name])
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

    def publish(self, from_host):
        if self.with_update:
            self.ctx.publish_weights(self.theta)
            self.version += 1
            if self.version % 1000 == 0:
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

    def step(self, events=None, e2e=False):
        torch = self.torch
        if events:
            events[0].record()
        self.actor()
        if events:
            events[1].record()
        self.learner()
        if events:
            events[2].record()
        self.publish(e2e)
        if e2e:
            if self.on_policy:
                self.host_adv_mean.copy_(self.adv[0, :1], non_blocking=True)
            else:
                self.host_td.copy_(self.out["td"], non_blocking=True)
                self.host_loss.copy_(self.out["loss"], non_blocking=True)
            torch.cuda.current_stream().synchronize()
        if events:
            events[3].record()

    def e2e_bytes(self):
        h2d = 0 if self.with_update else self.host_blobs[0].numel() * 4
        d2h = 4 if self.on_policy else (self.w["minibatch"] + 1) * 4
        return h2d, d2h


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
    w = synth.WORKLOADS[name]
    r = Runner(name, torch, binding, local, args.envs, args.with_update)
    w = r.w
    N = w["n_envs"]
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    ring_bytes = w["replay_capacity"] * (2 * w["obs_dim"] + 4) * 4
    need_flush = ring_bytes < 4 * (126 << 20)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        r.step()
    barrier()

    def timed_loop(K, e2e):
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
        launches0 = r.ctx.stats()["kernel_launches"]
        r.learner_ok = 0
        for i in range(K):
            if need_flush:
                flush.fill_(i & 0xFF)
            r.step(evs[i], e2e)
        torch.cuda.synchronize()
        tot = sum(e[0].elapsed_time(e[3]) for e in evs)
        act = sum(e[0].elapsed_time(e[1]) for e in evs)
        lrn = sum(e[1].elapsed_time(e[2]) for e in evs)
        return tot, act, lrn, r.ctx.stats()["kernel_launches"] - launches0, r.learner_ok

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    t_wall = time.time()
    tot_ms, act_ms, lrn_ms, launches, learner_ok = timed_loop(args.steps, False)
    barrier()
    wall = time.time() - t_wall
    clocks = sampler.stop() if rank == 0 else None
    e2e_ms, _, _, _, _ = timed_loop(args.steps, True)
    barrier()
    # the same K steps once more with the library's per-kernel CUDA events on: duration of each kernel class
    r.ctx.set_profiling(1)
    timed_loop(args.steps, False)
    prof = r.ctx.stats()
    r.ctx.set_profiling(0)
    barrier()

    tot_ms, e2e_ms, act_ms, lrn_ms = max_over_ranks([tot_ms, e2e_ms, act_ms, lrn_ms], "cuda")
    learner_ok = int(min_over_ranks([learner_ok], "cuda")[0])
    K = args.steps
    env_steps = N * r.actor_steps * K * world
    assert abs(aggregate_throughput(N * r.actor_steps * K, world, tot_ms) - env_steps / (tot_ms * 1e-3)) < 1e-6 * env_steps
    consumed = (w["rollout_len"] * N if r.on_policy else w["minibatch"]) * learner_ok * world
    value = env_steps / (tot_ms * 1e-3)
    flops, nbytes = actor_algorithmic(w)
    names = ["actor_fused", "mlp_tensor", "env_select_insert", "sample_gather", "td", "publish", "gae", "sgd_update"]
    kms, kcnt = prof["kernel_ms"], prof["kernel_count"]
    total_kms = sum(kms) or 1.0
    kernels = {names[i]: {"launches": kcnt[i], "ms": kms[i], "share": kms[i] / total_kms} for i in range(len(names)) if kcnt[i]}
    dom = max(range(len(names)), key=lambda i: kms[i])
    units = N * r.actor_steps                      # env-steps one actor call processes
    fma_peak = SM_COUNT * FMA_LANES_PER_SM * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12
    mlp_flops = 2 * mlp_macs(w)
    env_flops = flops - mlp_flops
    S_d = w["obs_dim"] if w["env_kind"] == synth.ENV_LINGAUSS else 4
    if dom == 1:      # tensor-core MLP: actor launches process N rows, learner launches B rows (two per step)
        rows = K * (r.actor_steps * N + 2 * w["minibatch"])
        achieved = mlp_flops * rows / (kms[1] * 1e-3) / 1e12
        roof = {"kernel": "actor_tc_pipelined_kernel (fused tcgen05 actor step; the TD forwards of mlp_bf16_tc_kernel share the class)",
                "bound": "tensor", "achieved": achieved,
                "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "peak_source": "cuBLAS bf16 sustained, of " + peaks["source"]}
    elif dom == 2:    # selection + env step + insert: state read twice (obs) + written, record written, outputs read
        per_env = 2 * S_d * 4 + 8 + (2 * w["obs_dim"] + 4) * 4 + w["n_actions"] * 4
        gbs = per_env * units * K / (kms[2] * 1e-3) / 1e9
        tfl = env_flops * units * K / (kms[2] * 1e-3) / 1e12
        if gbs / peaks["hbm_gbs"] >= tfl / fma_peak:
            roof = {"kernel": "actor_lingauss_kernel (selection + env step + insert)", "bound": "hbm", "achieved": gbs,
                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "peak_source": "copy bandwidth, of " + peaks["source"]}
        else:
            roof = {"kernel": "actor_lingauss_kernel (selection + env step + insert)", "bound": "alu", "achieved": tfl,
                    "peak": fma_peak, "unit": "TFLOP/s",
                    "peak_source": "FP32 FMA: 148 SMs x 128 lanes x 2 flop x max SM clock (derived, not measured)"}
    else:             # fused FP32 actor kernel (or, for tiny workloads, whatever dominates: reported against it)
        t_ms = kms[0] if kcnt[0] else act_ms
        achieved = flops * units * K / (t_ms * 1e-3) / 1e12
        roof = {"kernel": "actor_small_env_kernel (MLP + selection + env step + insert)", "bound": "alu",
                "achieved": achieved, "peak": fma_peak, "unit": "TFLOP/s",
                "peak_source": "FP32 FMA: 148 SMs x 128 lanes x 2 flop x max SM clock (derived, not measured)"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    per_env = NCU_DRAM_BYTES_PER_ENV_STEP.get(name) if dom == 1 else None
    roof["traffic"] = per_env * N if per_env else None
    roof["traffic_note"] = "bytes per fused actor launch (N env-steps), ncu capture at 113,664 envs scaled by N" if per_env else None
    roof["step_hbm_frac_of_measured"] = nbytes * units / (act_ms * 1e-3 / K) / 1e9 / peaks["hbm_gbs"]
    h2d, d2h = r.e2e_bytes()
    line = {
        "metric": "env-steps/s", "value": value, "unit": "env-steps/s", "n_gpus": world, "steps": K,
        "warmup": args.warmup, "ms_per_step": tot_ms / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w["weight_dtype"] == synth.W_BF16 else "f32", "data": "synthetic",
        "config": {"workload": name, "n_envs": N, "actor_steps_per_step": r.actor_steps,
                   "minibatch": w.get("minibatch"), "mlp": "%d-%d-%d-%d" % (w["obs_dim"], w["hidden"], w["hidden"], w["n_actions"]),
                   "replicas": world, "learner_update": r.with_update,
                   "l2": "flushed between steps (256 MiB write outside the per-step event pairs)" if need_flush
                   else "ring larger than L2"},
        "consumed_samples_per_s": consumed / (tot_ms * 1e-3),
        "actor_ms_per_step": act_ms / K, "learner_ms_per_step": lrn_ms / K, "wall_s": wall,
        "e2e": {"value": env_steps / (e2e_ms * 1e-3), "unit": "env-steps/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "roofline": roof,
        "kernels": kernels,
        "clocks": clocks,
    }
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(name, budget_s=args.cpu_seconds)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------- oracle arm
def oracle_sample_shape(name):
    """A bounded sample of the workload for the CPU oracle: fewer envs, the same call pattern."""
    w = synth.WORKLOADS[name]
    n_envs = {"cfg1": 64, "cfg2": 1024, "cfg3": 256, "cfg4": 256, "cfg5": 64}[name]
    n_envs = min(n_envs, w["n_envs"])
    over = dict(n_envs=n_envs)
    if w["replay_capacity"]:
        over["replay_capacity"] = n_envs * 64
        over["minibatch"] = min(w["minibatch"], 256)
        over["warmup"] = over["minibatch"]
    return over


def oracle_step_fn(name):
    import oracle
    w = synth.WORKLOADS[name]
    over = oracle_sample_shape(name)
    f = synth.config_fields(w, **over)
    o = oracle.Oracle(**f)
    vh = w["policy_kind"] == 1
    state = dict(v=0)
    on_policy = w["replay_capacity"] == 0
    a_steps = w["rollout_len"] if on_policy else w["actor_per_learner"]

    def publish():
        state["v"] += 1
        o.publish(synth.policy_blob(f["seed"], (state["v"] - 1) % 8 + 1, w["obs_dim"], w["hidden"], w["n_actions"], vh))

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
    desc = "%d of %d envs, %d actor steps + 1 learner step (minibatch %s) per step, single thread" % (
        f["n_envs"], w["n_envs"], a_steps, f.get("minibatch"))
    return step, desc


def cpu_baseline(name, budget_s=12.0):
    step, desc = oracle_step_fn(name)
    step()
    t0 = time.time()
    env_steps = consumed = n = 0
    while time.time() - t0 < budget_s:
        e, c = step()
        env_steps += e
        consumed += c
        n += 1
    dt = time.time() - t0
    return {"value": env_steps / dt, "unit": "env-steps/s", "cores": 1, "kind": "oracle",
            "sample": "%s; %d steps in %.1f s" % (desc, n, dt), "consumed_samples_per_s": consumed / dt}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.workload
    w = synth.WORKLOADS[name]
    step, desc = oracle_step_fn(name)
    for _ in range(args.warmup):
        step()
    t0 = time.time()
    env_steps = consumed = 0
    for _ in range(args.steps):
        e, c = step()
        env_steps += e
        consumed += c
    dt = time.time() - t0
    value = env_steps / dt
    line = {
        "impl": "reference", "metric": "env-steps/s", "value": value, "unit": "env-steps/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt * 1e3 / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": name, "n_envs": w["n_envs"], "sample": desc},
        "consumed_samples_per_s": consumed / dt,
        "cpu_baseline": {"value": value, "unit": "env-steps/s", "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "env-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="cfg5", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--envs", type=int, default=0, help="profiling aid: run the workload with this many envs (ring scaled to the same number of steps)")
    ap.add_argument("--with-update", action="store_true", help="FP32 replay workloads: the learner step also runs tj_sgd_step and publishes the parameters it trains")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
