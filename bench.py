#!/usr/bin/env python
"""Throughput of one PAAC iteration (rollout of t_max steps for n_e environments + one update)
on B200, reported as environment steps per second.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl ours|reference]

One "step" is one whole iteration of Algorithm 1 on the synthetic hashed environment.  The line
printed by rank 0 carries the device-timed value, an end-to-end figure through the
external-environment entry points (host frames in, actions out), a per-kernel CUDA-event breakdown
with a roofline entry for the kernel that takes the most time, and the CPU oracle timed on a
bounded sample of the same workload.  With --gpus N > 1 every rank runs an independent replica
(the path is single-GPU: environments are not sharded and nothing is exchanged).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1705_04862_b200.configs import COMMON, CONFIGS  # noqa: E402

FRAME_BYTES = 84 * 84 * 4
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of a kernel family from the ncu capture summarised
# under profiles/ (bytes); an entry is dropped when its kernel changes after the capture
NCU_TRAFFIC = {("cfg5_nature_bf16_ne1024", "conv1_fwd"): 29058560}


# ----------------------------------------------------------------------------- workload arithmetic
def net_layers(arch):
    """(name, rows per state, N, K) of each forward contraction."""
    if arch == "nips":
        return [("conv1", 400, 16, 256), ("conv2", 81, 32, 256), ("fc", 1, 256, 2592)], 256
    return [("conv1", 400, 32, 256), ("conv2", 81, 64, 512), ("conv3", 49, 64, 576), ("fc", 1, 512, 3136)], 512


def kernel_work(cfg):
    """Per kernel family: (roofline that bounds it, algorithmic FLOPs (2 x MAC, unpadded) or bytes of ONE logical
    launch, logical launches per iteration).  A logical launch may be more than one kernel (the fully
    connected forward is a split-k GEMM plus its finishing kernel).  Rollout kernels see n_e states per launch,
    update kernels B = n_e * t_max."""
    layers, F = net_layers(cfg["arch"])
    n_e, T, A = cfg["n_e"], cfg["t_max"], cfg["n_actions"]
    B = n_e * T
    elt = 2 if cfg["precision"] == "bf16" else 4
    P = sum(N * K + N for _, _, N, K in layers) + (A + 1) * (F + 1)
    w = {}
    for name, rows, N, K in layers:
        mac = rows * N * K
        w[name + "_fwd"] = ("tensor", 2.0 * mac * n_e, T + 1)
        w[name + "_wgrad"] = ("tensor", 2.0 * mac * B, 1)
        if name != "conv1":
            w[name + "_dgrad"] = ("tensor", 2.0 * mac * B, 1)
    w["heads_fwd_sample"] = ("tensor", 2.0 * (A + 1) * F * n_e, T + 1)
    w["heads_bwd"] = ("tensor", 4.0 * (A + 1) * F * B, 1)
    w["env_step"] = ("hbm", n_e * (FRAME_BYTES + 6.0), T)
    w["clip_rmsprop"] = ("hbm", P * (22.0 if elt == 2 else 20.0), 1)
    w["grad_sumsq"] = ("hbm", P * 4.0, 1)
    return w, P


def iteration_flops(cfg):
    layers, F = net_layers(cfg["arch"])
    A = cfg["n_actions"]
    fwd = sum(2.0 * r * N * K for _, r, N, K in layers) + 2.0 * (A + 1) * F
    bwd = 2.0 * fwd - 2.0 * layers[0][1] * layers[0][2] * layers[0][3]      # no data gradient for conv1
    n_e, T = cfg["n_e"], cfg["t_max"]
    return fwd * n_e * (T + 1), bwd * n_e * T


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sustained=d.get("bf16_tflops_sustained"),
                    src="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, src="fallback")


# ----------------------------------------------------------------------------- ranks
def max_over_ranks(x, dist=None, device="cpu"):
    """Largest value of x over the ranks of the job (x itself without a process group)."""
    if dist is None:
        return float(x)
    import torch
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank, world, ms_per_step):
    """Units all ranks processed per second, given the slowest rank's time per step (replicas: weak scaling)."""
    return world * units_per_rank / (ms_per_step * 1e-3)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t0, t1):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        rows = [r for ts, r in self.rows if t0 - 0.05 <= ts <= t1 + 0.15 and len(r) >= 7] or \
               [r for _, r in self.rows if len(r) >= 7]
        sm = sorted(float(r[0]) for r in rows if r[0].replace(".", "").isdigit())
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for j, n in enumerate(names) if any(r[3 + j].lower().startswith("active") for r in rows)]
        mx = [float(r[1]) for r in rows if r[1].replace(".", "").isdigit()]
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx[0] if mx else None,
                "reasons": reasons, "samples": len(rows)}


# ----------------------------------------------------------------------------- oracle legs
def oracle_time(cfg, n_e_sample, iters, warm=0):
    """Seconds per iteration of the CPU oracle on the first n_e_sample environments of cfg."""
    from oracle import oracle as orc
    orc.build()
    hp = dict(gamma=COMMON["gamma"], lr=cfg["lr"], rms_decay=COMMON["rms_decay"], rms_eps=COMMON["rms_eps"],
              clip_norm=COMMON["clip_norm"], entropy_beta=COMMON["entropy_beta"], value_coef=COMMON["value_coef"],
              term_denom=cfg["term_denom"])
    o = orc.OraclePAAC(cfg["arch"], n_e_sample, cfg["t_max"], cfg["n_actions"], COMMON["seed"],
                       bf16=cfg["precision"] == "bf16", hp=hp)
    for _ in range(warm):
        o.rollout()
        o.update()
    t0 = time.time()
    for _ in range(iters):
        o.rollout()
        o.update()
    return (time.time() - t0) / iters


def run_reference(args, cfg):
    """The oracle as it stands on the host cores; each step is one iteration on a bounded sample."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    cores = os.cpu_count() or 1
    total = max(1, args.steps + args.warmup)
    n_s = 1
    while n_s * 2 <= min(cfg["n_e"], 256) and 0.7 * n_s * 2 * total / max(cores, 1) <= 150:
        n_s *= 2
    sec = oracle_time(cfg, n_s, args.steps, warm=args.warmup)
    val = n_s * cfg["t_max"] / sec
    sample = "one iteration per step on the first %d of %d environments" % (n_s, cfg["n_e"])
    print(json.dumps({
        "impl": "reference", "metric": "env_steps_per_sec", "value": val, "unit": "env-steps/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg),
        "cpu_baseline": {"value": val, "unit": "env-steps/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "env-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def workload_config(cfg):
    return {"workload": cfg["name"], "arch": cfg["arch"], "precision": cfg["precision"], "n_e": cfg["n_e"],
            "t_max": cfg["t_max"], "n_actions": cfg["n_actions"], "update_batch": cfg["n_e"] * cfg["t_max"],
            "l2": "per-step working set (frames + stored activations) exceeds the 126 MB L2"
                  if cfg["n_e"] >= 256 else "working set fits L2; an L2-sized buffer is rewritten between steps"}


# ----------------------------------------------------------------------------- our arm
def run_ours(args, cfg):
    import torch
    from paper_1705_04862_b200 import binding as pb
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    hp = dict(gamma=COMMON["gamma"], lr=cfg["lr"], rms_decay=COMMON["rms_decay"], rms_eps=COMMON["rms_eps"],
              clip_norm=COMMON["clip_norm"], entropy_beta=COMMON["entropy_beta"], value_coef=COMMON["value_coef"],
              term_denom=cfg["term_denom"])
    prec = pb.BF16 if cfg["precision"] == "bf16" else pb.FP32
    # a stream of our own: the library records its launch sequences into CUDA graphs, which the legacy default
    # stream does not allow; every event below is recorded on this stream too
    side = torch.cuda.Stream()
    torch.cuda.set_stream(side)
    g = pb.Paac(cfg["arch"], cfg["n_e"], cfg["t_max"], cfg["n_actions"], COMMON["seed"] + rank, precision=prec,
                device="cuda:%d" % local, **hp)
    if args.fp32_tensor_cores:
        g.set_option(pb.OPT_FP32_TENSOR_CORES, 1)
    if args.update_chunks > 1:
        g.set_option(pb.OPT_UPDATE_CHUNKS, args.update_chunks)
    n_e, T = cfg["n_e"], cfg["t_max"]
    small = cfg["n_e"] < 256
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if small else None

    def step(sync_stats=False):
        if flush is not None:
            flush.zero_()
        g.rollout()
        return g.update(sync=sync_stats)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    # ---- timed region: K whole iterations, device time, max over ranks
    K = args.steps
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * K + 1)]
    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    l0, t0 = g.launch_count(), time.time()
    ev[0].record()
    for k in range(K):
        if flush is not None:
            flush.zero_()
        g.rollout()
        ev[2 * k + 1].record()
        g.update(sync=False)
        ev[2 * k + 2].record()
    barrier()
    t1 = time.time()
    launches = g.launch_count() - l0
    clocks = sampler.stop(t0, t1) if sampler else None
    total_ms = ev[0].elapsed_time(ev[2 * K])
    roll_ms = sum(ev[2 * k].elapsed_time(ev[2 * k + 1]) for k in range(K)) / K
    upd_ms = sum(ev[2 * k + 1].elapsed_time(ev[2 * k + 2]) for k in range(K)) / K
    total_ms = max_over_ranks(total_ms, dist, "cuda")
    ms_per_step = total_ms / K
    value = whole_job_value(n_e * T, world, ms_per_step)

    # ---- sustained block: the same iteration repeated for at least two seconds (how Algorithm 1 actually runs),
    # with the clocks sampled underneath; compare blocks by time x median SM MHz, not by a clock setting
    sustained = None
    if args.sustain_s > 0:
        sampler2 = ClockSampler(local) if rank == 0 else None
        barrier()
        s0 = time.time()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        n_sus, chunk = 0, max(50, int(0.25 / max(ms_per_step * 1e-3, 1e-6)))
        while True:
            for _ in range(chunk):
                if flush is not None:
                    flush.zero_()
                g.rollout()
                g.update(sync=False)
            n_sus += chunk
            torch.cuda.synchronize()
            if time.time() - s0 >= args.sustain_s:
                break
        e1.record()
        barrier()
        s1 = time.time()
        sus_ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda") / n_sus
        clk2 = sampler2.stop(s0, s1) if sampler2 else None
        sustained = {"ms_per_step": sus_ms, "steps": n_sus, "seconds": s1 - s0,
                     "value": whole_job_value(n_e * T, world, sus_ms), "clocks": clk2}

    # ---- per-kernel CUDA-event breakdown over another K steps (same kernels, event pairs around each)
    # Two passes, and for every family the faster of the two: one stalled launch (seen once: 2.9 ms on a 9 us kernel)
    # would otherwise decide which family counts as the dominant one.
    passes = []
    for _ in range(2):
        g.profile(True)
        for _ in range(K):
            step()
        passes.append(g.profile_read())
        g.profile(False)
    prof = {k: min((p[k] for p in passes if k in p), key=lambda v: v[0] / max(v[1], 1)) for k in passes[0]}

    # ---- the pre-processing kernel of Section 5.1 on n_e pairs of synthetic raw frames (bytes = two raw frames and the
    # previous state read, the new state written); the inputs (over 200 MB at n_e = 1024) exceed L2
    prep = None
    if rank == 0 and not args.no_e2e:
        raw = torch.randint(0, 256, (2, n_e, 210, 160, 3), dtype=torch.uint8, device="cuda")
        st_in = torch.randint(0, 256, (n_e, 84, 84, 4), dtype=torch.uint8, device="cuda")
        st_out = torch.empty_like(st_in)
        for _ in range(3):
            pb.preprocess(raw[0], raw[1], st_in, st_out, n_e, side.cuda_stream)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record()
        for _ in range(20):
            pb.preprocess(raw[0], raw[1], st_in, st_out, n_e, side.cuda_stream)
        p1.record()
        torch.cuda.synchronize()
        prep = {"ms": p0.elapsed_time(p1) / 20, "bytes": n_e * (2 * 210 * 160 * 3 + 2 * FRAME_BYTES)}
        del raw, st_in, st_out

    # ---- end to end through the external-environment entry points (host frames in, actions out)
    frames_dev = torch.empty(0)
    e2e = None
    if (rank == 0 or world > 1) and not args.no_e2e:
        g.rollout()
        import numpy as np
        fr = g.debug_read(pb.DBG_FRAMES).reshape(T, n_e, FRAME_BYTES)
        nx = g.debug_read(pb.DBG_NEXT_FRAMES).reshape(1, n_e, FRAME_BYTES)
        host_frames = torch.from_numpy(np.concatenate([fr, nx])).pin_memory()
        host_r = torch.from_numpy(g.debug_read(pb.DBG_REWARDS).reshape(T, n_e).copy()).pin_memory()
        host_t = torch.from_numpy(g.debug_read(pb.DBG_TERMINALS).reshape(T, n_e).copy()).pin_memory()
        host_a = torch.zeros(n_e, dtype=torch.int32).pin_memory()
        host_v = torch.zeros(n_e, dtype=torch.float32).pin_memory()
        g.update()

        host_planes = torch.from_numpy(np.ascontiguousarray(host_frames.numpy()[:, :, 3::4])).pin_memory()      # newest channel of every state

        def e2e_step(first=False, newest=True):
            # s_0 of an iteration is s_{t_max} of the one before (Algorithm 1) and already on the device: only the
            # first iteration sends it.  newest: every later state is built on the device from the one frame that
            # joins its four-frame stack (Section 5.1), a quarter of the bytes; else whole states are sent.
            for t in range(T):
                if t == 0 or not newest:
                    g.act_host(t, host_frames[t] if (first or t > 0) else None, host_a, host_v)
                else:
                    g.act_host_newest(t, host_planes[t], None, host_a, host_v)
                g.observe_host(t, host_r[t], host_t[t])
            if newest:
                g.act_host_newest(T, host_planes[T], None, None, host_v)
            else:
                g.act_host(T, host_frames[T], None, host_v)
            return g.update(sync=True)

        Ke = max(3, min(K, 10))
        timed = {}
        for newest in (False, True):
            e2e_step(first=True, newest=newest)
            e2e_step(newest=newest)
            barrier()
            w0 = time.time()
            for _ in range(Ke):
                e2e_step(newest=newest)
            barrier()
            timed[newest] = max_over_ranks((time.time() - w0) / Ke, dist, "cuda")
        e_sec = timed[True]
        plane_bytes = n_e * (FRAME_BYTES // 4)
        e2e = {"value": whole_job_value(n_e * T, world, e_sec * 1e3), "unit": "env-steps/s", "ms_per_step": e_sec * 1e3,
               "h2d_bytes_per_step": T * plane_bytes + 2 * T * n_e,
               "d2h_bytes_per_step": T * n_e * 4 + (T + 1) * n_e * 4 + 32,
               "api": "paac_act_host (step 0, taken from the device) / paac_act_host_newest (one new 84 x 84 frame per "
                      "environment and step; the four-frame state is assembled on the device) / paac_observe_host / "
                      "paac_update, pinned host buffers, wall clock",
               "whole_states": {"value": whole_job_value(n_e * T, world, timed[False] * 1e3), "ms_per_step": timed[False] * 1e3,
                                "h2d_bytes_per_step": T * n_e * FRAME_BYTES + 2 * T * n_e,
                                "api": "paac_act_host with whole 84 x 84 x 4 states for steps 1 .. t_max"}}
    del frames_dev
    g.close()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the kernel family that takes the most time
    pk = peaks()
    work, P = kernel_work(cfg)
    tot = sum(ms for ms, _ in prof.values())
    shares = {k: {"ms_per_step": ms / K, "launches_per_step": n / K, "share": ms / tot} for k, (ms, n) in prof.items()}
    dom = max((k for k in prof if k in work and work[k][1] > 0), key=lambda k: prof[k][0])
    bound, amount, logical = work[dom]
    dom_ms = prof[dom][0] / K / logical                    # device time of one logical launch
    if bound == "tensor":
        ach, peak, unit = amount / (dom_ms * 1e-3) / 1e12, pk["bf16"], "TFLOP/s"
    else:
        ach, peak, unit = amount / (dom_ms * 1e-3) / 1e9, pk["hbm"], "GB/s"
    roll_flops, upd_flops = iteration_flops(cfg)
    upd_tflops = upd_flops / (upd_ms * 1e-3) / 1e12
    roofline = {"kernel": dom, "bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                "traffic": NCU_TRAFFIC.get((cfg["name"], dom)), "peak_source": pk["src"], "avg_launch_ms": dom_ms,
                "algorithmic_per_launch": amount,
                # the whole update (all backward kernels, stored activations reused) against the tensor peaks
                "update_ms": upd_ms, "update_tflops": upd_tflops, "update_frac_of_bf16_peak": upd_tflops / pk["bf16"],
                "update_frac_of_bf16_sustained": upd_tflops / pk["bf16_sustained"] if pk.get("bf16_sustained") else None,
                "iteration_frac_of_bf16_peak": (roll_flops + upd_flops) / (ms_per_step * 1e-3) / 1e12 / pk["bf16"]}
    if sustained is not None:
        # the update's share of an iteration is taken from the burst block (events inside the long block would stall it)
        sus_upd_ms = sustained["ms_per_step"] * upd_ms / (roll_ms + upd_ms)
        sustained["update_frac_of_bf16_sustained"] = (upd_flops / (sus_upd_ms * 1e-3) / 1e12 / pk["bf16_sustained"]
                                                      if pk.get("bf16_sustained") else None)
        sustained["iteration_tflops"] = (roll_flops + upd_flops) / (sustained["ms_per_step"] * 1e-3) / 1e12
    hbm_side = {}
    for k in ("env_step", "clip_rmsprop", "grad_sumsq"):
        if k in prof and prof[k][1]:
            gbs = work[k][1] / (prof[k][0] / K / work[k][2] * 1e-3) / 1e9
            hbm_side[k] = {"GB/s": gbs, "frac_of_%s_hbm" % pk["src"]: gbs / pk["hbm"]}
    if prep is not None:
        gbs = prep["bytes"] / (prep["ms"] * 1e-3) / 1e9
        hbm_side["preprocess"] = {"GB/s": gbs, "frac_of_%s_hbm" % pk["src"]: gbs / pk["hbm"], "ms": prep["ms"],
                              "note": "20 back-to-back launches on n_e raw frame pairs"}
    per_family = {}
    for k, (ms, n) in prof.items():
        if k in work and work[k][0] == "tensor":
            per_family[k] = work[k][1] * work[k][2] / (ms / K * 1e-3) / 1e12
    # ---- CPU oracle on a bounded sample (rank 0, one GPU only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cores = os.cpu_count() or 1
        n_s = min(cfg["n_e"], 128 if cfg["arch"] == "nature" else 512)
        sec = oracle_time(cfg, n_s, 1)
        cpu = {"value": n_s * T / sec, "unit": "env-steps/s", "cores": cores, "kind": "oracle",
               "sample": "one iteration on the first %d of %d environments (%.1f s)" % (n_s, cfg["n_e"], sec)}

    out = {
        "metric": "env_steps_per_sec", "value": value, "unit": "env-steps/s", "n_gpus": world, "steps": K,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg["precision"], "data": "synthetic",
        "config": dict(workload_config(cfg), **({"contractions": "3xTF32 tensor cores"} if args.fp32_tensor_cores else {}),
                       **({"update_chunks": args.update_chunks} if args.update_chunks > 1 else {})),
        "updates_per_sec": world * 1e3 / ms_per_step, "rollout_ms": roll_ms, "update_ms": upd_ms,
        "rollout_tflops": roll_flops / (roll_ms * 1e-3) / 1e12,
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "sustained": sustained,
        "cpu_baseline": cpu, "hbm_kernels": hbm_side,
        # per-kernel pass: plain launches with an event pair around each, so every figure carries a launch gap the
        # timed region (CUDA graphs, dependent launches) does not have: the sum exceeds ms_per_step
        "kernels_sum_ms": tot / K, "kernels_note": "plain launches with event pairs; sum exceeds ms_per_step by the launch gaps",
        "kernel_tflops": per_family, "kernels": shares,
    }
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def run_lr_sweep(args):
    """Section 5.3's learning-rate rule, alpha = 0.0007 * n_e for n_e in 16 .. 256, on the learnable synthetic
    environment (a bright band of rows names the rewarded action; chance level 1 / A): mean reward per step at the
    start and at the end of a fixed budget of timesteps, and where training stopped being finite if it did.
    The environment is a contextual bandit (the next state's goal does not depend on the action), so the sweep runs
    with gamma = 0: the one-step return is then the exact advantage target, and the value head predicts a quantity
    of order one as it does under the clipped, sparse rewards of the paper's games (with gamma = 0.99 a reward on
    every step makes the value targets of order 1 / (1 - gamma) and the paper's step sizes collapse the policy).
    All other hyper-parameters are Section 5.1's."""
    import numpy as np
    import torch
    from paper_1705_04862_b200 import binding as pb
    torch.cuda.set_stream(torch.cuda.Stream())
    A, T, budget = 6, 5, args.sweep_timesteps
    rows = []
    for arch, prec in (("nips", pb.FP32), ("nature", pb.BF16)):
        for n_e in (16, 32, 64, 128, 256):
            lr = 0.0007 * n_e
            g = pb.Paac(arch, n_e, T, A, COMMON["seed"], precision=prec, lr=lr, term_denom=200, environment=pb.ENV_PATTERN,
                        gamma=0.0, rms_decay=COMMON["rms_decay"], rms_eps=COMMON["rms_eps"],
                        clip_norm=COMMON["clip_norm"], entropy_beta=COMMON["entropy_beta"], value_coef=COMMON["value_coef"])
            updates = max(40, budget // (n_e * T))
            rew, ent, bad = [], [], None
            for u in range(updates):
                g.rollout()
                rew.append(float(g.debug_read(pb.DBG_REWARDS).astype(np.float64).mean()))
                st = g.update()
                ent.append(st["entropy"])
                if st["status"] != 0 and bad is None:
                    bad = u
            k = max(5, updates // 10)
            above = [i for i in range(len(rew) - 4) if np.mean(rew[i:i + 5]) >= 0.8]
            rows.append({"arch": arch, "precision": "bf16" if prec == pb.BF16 else "fp32", "n_e": n_e, "lr": lr,
                         "updates": updates, "timesteps": updates * n_e * T, "reward_first": float(np.mean(rew[:k])),
                         "reward_last": float(np.mean(rew[-k:])), "entropy_last": float(np.mean(ent[-k:])),
                         "timesteps_to_0.8": (above[0] + 5) * n_e * T if above else None, "first_nonfinite_update": bad})
            g.close()
    print(json.dumps({"experiment": "lr_rule_sweep", "rule": "lr = 0.0007 * n_e", "environment": "pattern", "n_actions": A,
                      "t_max": T, "gamma": 0.0, "chance_reward": 1.0 / A, "rows": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=4, help="index into the five workloads (4 = n_e 1024, Nature CNN, bf16)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true",
                    help="skip the end-to-end leg and the pre-processing kernel (short runs under a profiler)")
    ap.add_argument("--sustain-s", type=float, default=2.0,
                    help="seconds of back-to-back iterations in the sustained block (0 = skip it)")
    ap.add_argument("--fp32-tensor-cores", action="store_true",
                    help="float configurations: every contraction as three TF32 tensor-core passes (float-accurate)")
    ap.add_argument("--update-chunks", type=int, default=1,
                    help="bf16 configurations: conv2 data gradient / conv1 weight gradient over this many groups of states")
    ap.add_argument("--lr-sweep", action="store_true",
                    help="instead of the throughput line: the alpha = 0.0007 n_e rule on the learnable environment")
    ap.add_argument("--sweep-timesteps", type=int, default=200000)
    args = ap.parse_args()
    cfg = CONFIGS[args.config]
    if args.lr_sweep:
        run_lr_sweep(args)
        return
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
