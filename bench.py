#!/usr/bin/env python
"""Benchmark of the dense 3x3x3 conv3d passes (forward, data gradient, weight gradient).

Workload: the single-layer sweep - NDHWC bf16, batch 1, 128x128x128 volume, 3x3x3 stride 1
pad 1, C_in = C_out in {32, 64, 128, 256}, activations and upstream gradients N(0,1), Kaiming
weights, seed 2.  One step = forward + dgrad + wgrad for every channel count.  The metric is
dense FLOP/s: 2 * 27 * C^2 * voxels per pass (padded taps counted).

    python bench.py --gpus 1 --steps 5 --warmup 3
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N   (independent replicas)
    python bench.py --impl reference     (the CPU oracle on a bounded sample, same metric)

Prints one JSON line.
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

CHANNELS = (32, 64, 128, 256)
VOL = (128, 128, 128)
SEED = 2
NOMINAL_BF16_TFLOPS = 2250.0
PROFILES = os.path.join(ROOT, "profiles")


def ncu_traffic_bytes(summary, sources):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch, as recorded in a profiles/ summary: the line
    `traffic_bytes_per_launch: <bytes>`.  The summary also records `source_sha256: <hex>` of the kernel's source
    files at the time of the capture; when the files differ today the counters no longer describe the kernel and
    the answer is None."""
    import hashlib
    try:
        text = open(os.path.join(PROFILES, summary)).read()
    except OSError:
        return None
    val = sha = None
    for line in text.splitlines():
        if line.startswith("traffic_bytes_per_launch:"):
            val = float(line.split(":", 1)[1].split()[0])
        elif line.startswith("source_sha256:"):
            sha = line.split(":", 1)[1].split()[0]
    h = hashlib.sha256()
    try:
        for f in sources:
            h.update(open(os.path.join(ROOT, "paper_2006_12575_b200", "csrc", f), "rb").read())
    except OSError:
        return None
    return val if (val is not None and sha == h.hexdigest()) else None


def pass_flops(C, vol=VOL):
    return 2.0 * 27 * C * C * vol[0] * vol[1] * vol[2]


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return dict(hbm_gbs=float(d["hbm_gbs"]), bf16=float(d["bf16_tflops"]),
                        bf16_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
        except Exception:
            pass
    return dict(hbm_gbs=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


# --------------------------------------------------------------------------------------------
# CPU oracle legs (cpu_baseline of the GPU arm, and the whole of --impl reference)
# --------------------------------------------------------------------------------------------
ORACLE_SAMPLE = dict(C=64, slab=(16, 64, 64))
CPU_BASELINE_REPEATS = 3


def oracle_sample_once():
    """fwd + dgrad + wgrad of the oracle on a slab of the workload.  Returns (seconds, flops)."""
    from oracle import ops
    from paper_2006_12575_b200 import synth
    C = ORACLE_SAMPLE["C"]
    D, H, W = ORACLE_SAMPLE["slab"]
    x = synth.normal_bf16((1, D, H, W, C), SEED).astype(np.float64)
    dy = synth.normal_bf16((1, D, H, W, C), SEED + 1).astype(np.float64)
    w = synth.kaiming_bf16(27, C, C, 27 * C, SEED + 2).astype(np.float64)
    t0 = time.perf_counter()
    ops.conv3d_fwd(x, w, None, 3, 1, 1)
    ops.conv3d_dgrad(dy, w, (D, H, W), 3, 1, 1)
    ops.conv3d_wgrad(x, dy, 3, 1, 1)
    return time.perf_counter() - t0, 3 * pass_flops(C, (D, H, W))


def oracle_description():
    from oracle import ops
    D, H, W = ORACLE_SAMPLE["slab"]
    return dict(kind="oracle", cores=ops.n_threads(), unit="TFLOP/s",
                sample=f"fwd+dgrad+wgrad, C={ORACLE_SAMPLE['C']}, 1x{D}x{H}x{W} slab of the 128^3 volume, fp64 direct loops")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import ops
    ops.build()
    for _ in range(min(args.warmup, 1)):
        oracle_sample_once()
    secs, flops = 0.0, 0.0
    steps = max(1, min(args.steps, 3))
    for _ in range(steps):
        s, f = oracle_sample_once()
        secs += s
        flops += f
    val = flops / secs / 1e12
    desc = oracle_description()
    desc["value"] = val
    out = dict(impl="reference", metric="conv3d_tflops", value=val, unit="TFLOP/s", n_gpus=args.gpus, steps=steps,
               warmup=min(args.warmup, 1), ms_per_step=1e3 * secs / steps, higher_is_better=True, scaling="weak",
               vs_baseline=None, dtype="f64", data="synthetic",
               config=dict(workload="conv3d sweep 128^3, C=32/64/128/256, fwd+dgrad+wgrad (bounded sample per step)"),
               cpu_baseline=desc, e2e=dict(value=val, unit="TFLOP/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(out), flush=True)


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc = None
        self.path = f"/tmp/lamp_bench_clocks_{os.getpid()}.csv"
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        res = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if not self.proc:
            return res
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if sm:
            res = dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return res


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2006_12575_b200 import binding as B
    from paper_2006_12575_b200 import build as lamp_build
    from paper_2006_12575_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        lamp_build.build()
    if world > 1:
        dist.barrier()
    B.lib()
    chans = tuple(int(c) for c in args.channels.split(","))
    D, H, W = VOL
    dev = torch.device("cuda", local)

    # host (pinned) copies of every input, device buffers for inputs and outputs
    host, devb = {}, {}
    for C in chans:
        g = torch.Generator().manual_seed(SEED * 1000 + C + 7919 * rank)
        hx = torch.randn((1, D, H, W, C), generator=g, dtype=torch.float32).to(torch.bfloat16).pin_memory()
        hdy = torch.randn((1, D, H, W, C), generator=g, dtype=torch.float32).to(torch.bfloat16).pin_memory()
        hw = torch.from_numpy(synth.kaiming_bf16(27, C, C, 27 * C, SEED * 1000 + C)).to(torch.bfloat16).pin_memory()
        host[C] = (hx, hdy, hw)
        desc = B.conv_desc(C, C)
        x = hx.to(dev)
        wsz = max(B.lamp_conv3d_workspace_bytes(desc, x, B.PASS_DGRAD), B.lamp_conv3d_workspace_bytes(desc, x, B.PASS_WGRAD), 256)
        devb[C] = dict(desc=desc, x=x, dy=hdy.to(dev), w=hw.to(dev), y=torch.empty_like(x), dx=torch.empty_like(x),
                       dw=torch.empty((27, C, C), dtype=torch.float32, device=dev),
                       ws=torch.empty(wsz, dtype=torch.uint8, device=dev))
    hout = {C: (torch.empty((1, D, H, W, C), dtype=torch.bfloat16).pin_memory(),
                torch.empty((1, D, H, W, C), dtype=torch.bfloat16).pin_memory(),
                torch.empty((27, C, C), dtype=torch.float32).pin_memory()) for C in chans}

    ev = lambda: torch.cuda.Event(enable_timing=True)
    pass_events = []

    def step(record):
        for C in chans:
            b = devb[C]
            marks = [ev() for _ in range(4)] if record else None
            if record:
                marks[0].record()
            B.lamp_conv3d_fwd(b["desc"], b["x"], b["w"], None, b["y"])
            if record:
                marks[1].record()
            B.lamp_conv3d_dgrad(b["desc"], b["dy"], b["w"], b["dx"], b["ws"])
            if record:
                marks[2].record()
            B.lamp_conv3d_wgrad(b["desc"], b["x"], b["dy"], b["dw"], None, b["ws"])
            if record:
                marks[3].record()
                pass_events.append((C, marks))

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step(False)
    sync_all()
    sampler = ClockSampler(local) if rank == 0 else None
    t0, t1 = ev(), ev()
    t0.record()
    for _ in range(args.steps):
        step(True)
    t1.record()
    sync_all()
    ms = t0.elapsed_time(t1)
    clocks = sampler.stop() if sampler else None
    status = B.lamp_get_async_status()
    if status != 0:
        raise SystemExit(f"bench.py: device status {status}")

    # The same passes once more, one channel count at a time (its three passes repeated back to back).  In the step above
    # the narrow layers' 2 ms follow 15 ms of C = 256 at the power cap and inherit that phase's SM clock; here every
    # channel count runs at the clock its own load settles at.  Reported beside `passes`, not instead of it.
    alone_events = []
    for C in chans:
        b = devb[C]
        # about 40 ms of untimed repetitions first: the SM clock needs that long to settle after the step above
        est_ms = sum(3 * pass_flops(C) for _ in (0,)) / 1.0e15 * 1e3
        warm = max(3, int(40.0 / max(est_ms, 1e-3)))
        for it in range(warm + 10):
            marks = [ev() for _ in range(4)]
            marks[0].record()
            B.lamp_conv3d_fwd(b["desc"], b["x"], b["w"], None, b["y"])
            marks[1].record()
            B.lamp_conv3d_dgrad(b["desc"], b["dy"], b["w"], b["dx"], b["ws"])
            marks[2].record()
            B.lamp_conv3d_wgrad(b["desc"], b["x"], b["dy"], b["dw"], None, b["ws"])
            marks[3].record()
            if it >= warm:
                alone_events.append((C, marks))
    sync_all()

    # end to end through the same calls with host buffers: H2D of x, dy, w and D2H of y, dx, dw every step.
    # Copies run on their own streams so that the transfers of one channel count overlap the kernels of another.
    cur = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = {C: torch.cuda.Event() for C in chans}
    ev_comp = {C: torch.cuda.Event() for C in chans}
    ev_out = {C: torch.cuda.Event() for C in chans}
    for C in chans:
        ev_comp[C].record(cur)
        ev_out[C].record(cur)

    def e2e_step():
        for C in chans:
            b = devb[C]
            hx, hdy, hw = host[C]
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_comp[C])              # the previous step no longer reads these inputs
                b["x"].copy_(hx, non_blocking=True)
                b["dy"].copy_(hdy, non_blocking=True)
                b["w"].copy_(hw, non_blocking=True)
                ev_in[C].record(s_in)
            cur.wait_event(ev_in[C])
            cur.wait_event(ev_out[C])                    # the previous step's results have left the device buffers
            B.lamp_conv3d_fwd(b["desc"], b["x"], b["w"], None, b["y"])
            B.lamp_conv3d_dgrad(b["desc"], b["dy"], b["w"], b["dx"], b["ws"])
            B.lamp_conv3d_wgrad(b["desc"], b["x"], b["dy"], b["dw"], None, b["ws"])
            ev_comp[C].record(cur)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_comp[C])
                hout[C][0].copy_(b["y"], non_blocking=True)
                hout[C][1].copy_(b["dx"], non_blocking=True)
                hout[C][2].copy_(b["dw"], non_blocking=True)
                ev_out[C].record(s_out)

    def e2e_drain():
        for C in chans:
            cur.wait_event(ev_out[C])
            cur.wait_event(ev_in[C])

    e2e_step()
    e2e_drain()
    sync_all()
    e0, e1 = ev(), ev()
    e2e_steps = max(1, min(args.steps, 3))
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e2e_drain()
    e1.record()
    sync_all()
    e2e_ms = e0.elapsed_time(e1)

    from paper_2006_12575_b200 import replicas
    ms, e2e_ms = replicas.job_time_ms(ms, dev), replicas.job_time_ms(e2e_ms, dev)       # slowest rank

    flops_step = sum(3 * pass_flops(C) for C in chans)
    value = world * flops_step * args.steps / (ms * 1e-3) / 1e12
    e2e_val = world * flops_step * e2e_steps / (e2e_ms * 1e-3) / 1e12
    h2d = sum(2 * D * H * W * C * 2 + 27 * C * C * 2 for C in chans)
    d2h = sum(2 * D * H * W * C * 2 + 27 * C * C * 4 for C in chans)

    # per-pass times (this rank), and the roofline of the kernel with the largest share
    per = {}
    for C, m in pass_events:
        for name, a, b_ in (("fwd", m[0], m[1]), ("dgrad", m[1], m[2]), ("wgrad", m[2], m[3])):
            per.setdefault((C, name), []).append(a.elapsed_time(b_))
    peaks = measured_peaks()
    passes = {}
    for (C, name), v in per.items():
        mean = sum(v) / len(v)
        tf = pass_flops(C) / (mean * 1e-3) / 1e12
        passes[f"C{C}.{name}"] = dict(ms=round(mean, 4), tflops=round(tf, 1), pct_nominal=round(100 * tf / NOMINAL_BF16_TFLOPS, 1),
                                      pct_measured=round(100 * tf / peaks["bf16"], 1))
    per_alone = {}
    for C, m in alone_events:
        for name, a, b_ in (("fwd", m[0], m[1]), ("dgrad", m[1], m[2]), ("wgrad", m[2], m[3])):
            per_alone.setdefault((C, name), []).append(a.elapsed_time(b_))
    passes_alone = {}
    for (C, name), v in per_alone.items():
        mean = sum(v) / len(v)
        tf = pass_flops(C) / (mean * 1e-3) / 1e12
        passes_alone[f"C{C}.{name}"] = dict(ms=round(mean, 4), tflops=round(tf, 1), pct_nominal=round(100 * tf / NOMINAL_BF16_TFLOPS, 1))
    # kernel families (one CUDA kernel template each); the dgrad pass also holds the tiny weight-transpose launch
    cmax = max(chans)
    # (C >= 128: conv3_t_kernel; C = 64: conv3_r_kernel)
    fwd_name = "conv3_t_kernel" if cmax >= 128 else "conv3_r_kernel" if cmax == 64 else "conv3_t_kernel"
    traffic_of = {f"{fwd_name} (fwd+dgrad, C={cmax})": ("conv3_t_c256_128cube.txt", ["conv_t.cu", "umma_ptx.cuh"]) if cmax == 256 else
                  ("conv3_r_c64_128cube.txt", ["conv_r.cu", "umma_ptx.cuh"]) if cmax == 64 else None,
                  f"wgrad_win_kernel (wgrad, C={cmax})": ("wgrad_win_c256_128cube.txt", ["wgrad_win.cu", "umma_ptx.cuh"]) if cmax == 256 else None}
    fam = {f"{fwd_name} (fwd+dgrad, C={cmax})": [k for k in per if k[1] in ("fwd", "dgrad") and k[0] == cmax],
           f"conv3_t_kernel / conv3_r_kernel (fwd+dgrad, C<{cmax})": [k for k in per if k[1] in ("fwd", "dgrad") and k[0] != cmax],
           f"wgrad_win_kernel (wgrad, C={cmax})": [k for k in per if k[1] == "wgrad" and k[0] == cmax],
           f"wgrad_win_kernel (wgrad, C<{cmax})": [k for k in per if k[1] == "wgrad" and k[0] != cmax]}
    fam = {f: ks for f, ks in fam.items() if ks}
    fam_time = {f: sum(sum(per[k]) for k in ks) for f, ks in fam.items()}
    dom = max(fam_time, key=fam_time.get)
    dom_flops = sum(pass_flops(k[0]) * len(per[k]) for k in fam[dom])
    dom_launches = sum(len(per[k]) for k in fam[dom])
    achieved = dom_flops / (fam_time[dom] * 1e-3) / 1e12
    roofline = dict(bound="tensor", kernel=dom, achieved=round(achieved, 2), peak=peaks["bf16"], unit="TFLOP/s",
                    frac=round(achieved / peaks["bf16"], 4),
                    traffic=ncu_traffic_bytes(*traffic_of[dom]) if traffic_of.get(dom) else None,
                    peak_source=peaks["source"] + " cuBLAS bf16 burst", frac_of_nominal_2250=round(achieved / NOMINAL_BF16_TFLOPS, 4),
                    algorithmic_flops_per_launch=dom_flops / dom_launches,
                    avg_launch_ms=round(fam_time[dom] / dom_launches, 4),
                    share_of_step=round(fam_time[dom] / sum(fam_time.values()), 3),
                    family_shares={f: round(t / sum(fam_time.values()), 3) for f, t in fam_time.items()})

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = oracle_description()
    try:
        from oracle import ops
        ops.build()
        secs, fl = 0.0, 0.0
        for _ in range(CPU_BASELINE_REPEATS):          # about 10 s of CPU work in all
            s_, f_ = oracle_sample_once()
            secs += s_
            fl += f_
        cpu["value"] = fl / secs / 1e12
        cpu["seconds"] = round(secs, 2)
        cpu["sample"] += f", {CPU_BASELINE_REPEATS} repetitions"
    except Exception as e:       # the baseline leg must not take the GPU numbers down with it
        cpu["value"] = None
        cpu["error"] = str(e)[:200]

    # the U-Net half of the metric, in the same process right after the sweep (one replica only: these workloads
    # hold up to 31 GB and are quoted per GPU): training step of the standard network, whole-volume against
    # sliding-window inference on the 512 x 512 x 128 volume
    unet = None
    if world == 1 and not args.no_unet:
        del devb, host, hout
        torch.cuda.empty_cache()
        unet = {}
        for key, wl, cfg_id, st_, wu_ in (("train_step_configs2", "unet_train", 2, 10, 3),
                                          ("whole_volume_configs4", "unet_infer", 4, 5, 3),
                                          ("sliding_window_configs4", "sliding", 4, 3, 3)):
            smp = ClockSampler(local)
            try:
                r = measure_unet(wl, cfg_id, st_, wu_, args.sw_batch, graph=False)
                r = {k: r[k] for k in ("metric", "value", "unit", "ms_per_step", "seconds_per_volume", "tflops", "steps", "warmup",
                                       "config", "roofline")}
            except Exception as e:                       # must not take the headline down with it
                r = dict(error=str(e)[:200])
            r["clocks"] = smp.stop()
            unet[key] = r
            torch.cuda.empty_cache()
        a, b_ = unet.get("whole_volume_configs4", {}), unet.get("sliding_window_configs4", {})
        if "seconds_per_volume" in a and "seconds_per_volume" in b_:
            unet["whole_volume_speedup_over_sliding_window"] = round(b_["seconds_per_volume"] / a["seconds_per_volume"], 2)

    launches_per_C = 1 + 2 + 2     # fwd; dgrad = weight transpose + conv; wgrad = split-K kernel + fixed-order reduce
    out = dict(metric="conv3d_tflops", value=round(value, 3), unit="TFLOP/s", n_gpus=world, steps=args.steps,
               warmup=args.warmup, ms_per_step=round(ms / args.steps, 4), higher_is_better=True, scaling="weak",
               vs_baseline=None, dtype="bf16", data="synthetic",
               config=dict(workload="configs[1]: conv3d 3x3x3 s1 p1 sweep, NDHWC bf16, 1x128x128x128, C_in=C_out in "
                                    + "/".join(str(c) for c in chans) + ", fwd+dgrad+wgrad per C",
                           l2="inputs larger than L2: a step streams several GB through distinct buffers",
                           flops_convention="2*27*C^2*voxels per pass", replicas=world),
               clocks=clocks,
               e2e=dict(value=round(e2e_val, 3), unit="TFLOP/s", h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                        steps=e2e_steps),
               gpu_launches=args.steps * len(chans) * launches_per_C,
               roofline=roofline, cpu_baseline=cpu, passes=passes,
               passes_one_channel_count_at_a_time=passes_alone,
               pct_of_nominal_bf16=round(100 * value / world / NOMINAL_BF16_TFLOPS, 2))
    if unet is not None:
        out["unet"] = unet
    print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------
# Secondary workloads: the U-Net passes (one JSON line each; the headline stays the conv sweep)
# --------------------------------------------------------------------------------------------
UNET_CFGS = {
    0: dict(levels=3, ch=[8, 16, 32], cpl=2, K=4, vol=(32, 32, 32)),
    2: dict(levels=5, ch=[32, 64, 128, 256, 512], cpl=2, K=10, vol=(128, 128, 128)),
    3: dict(levels=5, ch=[64, 128, 256, 512, 1024], cpl=3, K=10, vol=(192, 192, 64)),
    4: dict(levels=5, ch=[32, 64, 128, 256, 512], cpl=2, K=10, vol=(512, 512, 128)),
}


def unet_fwd_flops(cfg):
    D, H, W = cfg["vol"]
    ch, L = cfg["ch"], cfg["levels"]
    vox = [(D >> l) * (H >> l) * (W >> l) for l in range(L)]
    fl, c = 0.0, 1
    for l in range(L):
        for _ in range(cfg["cpl"]):
            fl += 2.0 * 27 * c * ch[l] * vox[l]
            c = ch[l]
        if l < L - 1:
            fl += 2.0 * 27 * ch[l] * ch[l + 1] * vox[l + 1]
            c = ch[l + 1]
    for l in range(L - 2, -1, -1):
        fl += 2.0 * ch[l + 1] * ch[l] * vox[l]
        c = 2 * ch[l]
        for _ in range(cfg["cpl"]):
            fl += 2.0 * 27 * c * ch[l] * vox[l]
            c = ch[l]
    return fl + 2.0 * ch[0] * cfg["K"] * vox[0]


def unet_floor_ms(cfg, train, peaks, vol=None, probs_out=True):
    """Roofline floor of one U-Net pass: the sum over its steps of max(FLOPs / tensor peak, algorithmic bytes /
    HBM peak), with the measured peaks.  Bytes per step: a conv reads its input and writes its output once
    (bf16) and reads its weights; normalise + ReLU moves 4 B per element; its backward 10 B per element; a data
    gradient reads dy and writes dx; a weight gradient reads x and dy and writes fp32 weights; the head reads
    its input and writes K fp32 probabilities and one label per voxel (training: reads them again and writes
    the gradient of its input)."""
    D, H, W = vol or cfg["vol"]
    ch, L, K = cfg["ch"], cfg["levels"], cfg["K"]
    vox = [(D >> l) * (H >> l) * (W >> l) for l in range(L)]
    tf, bw = peaks["bf16"] * 1e12, peaks["hbm_gbs"] * 1e9
    total = 0.0

    def step(flops, nbytes):
        nonlocal total
        total += max(flops / tf, nbytes / bw)

    def conv(ci, co, vin, vout, taps, norm, dgrad=True):
        fl = 2.0 * taps * ci * co * vout
        io = 2.0 * vin * ci + 2.0 * vout * co
        step(fl, io + 2.0 * taps * ci * co)
        if norm:
            step(0, 4.0 * vout * co)
        if train:
            if norm:
                step(0, 10.0 * vout * co)
            if dgrad:
                step(fl, io + 2.0 * taps * ci * co)
            step(fl, io + 4.0 * taps * ci * co)

    c = 1
    for l in range(L):
        for i in range(cfg["cpl"]):
            conv(c, ch[l], vox[l], vox[l], 27, True, dgrad=not (l == 0 and i == 0))
            c = ch[l]
        if l < L - 1:
            conv(ch[l], ch[l + 1], vox[l], vox[l + 1], 27, True)
            c = ch[l + 1]
    for l in range(L - 2, -1, -1):
        # transposed conv: one tap per output voxel
        fl = 2.0 * ch[l + 1] * ch[l] * vox[l]
        io = 2.0 * vox[l + 1] * ch[l + 1] + 2.0 * vox[l] * ch[l]
        step(fl, io)
        if train:
            step(fl, io)
            step(fl, io)
        c = 2 * ch[l]
        for _ in range(cfg["cpl"]):
            conv(c, ch[l], vox[l], vox[l], 27, True)
            c = ch[l]
    step(2.0 * ch[0] * K * vox[0], vox[0] * (2.0 * ch[0] + (4.0 * K if probs_out else 0.0) + 1))
    if train:
        step(4.0 * ch[0] * K * vox[0], vox[0] * (4.0 * ch[0] + 4.0 * K + 1))
    return total * 1e3


_VOLUMES = {}


def measure_unet(workload, cfg_id, steps, warmup, sw_batch=32, graph=True, se_ratio=0):
    """Times one U-Net workload on cuda:0 through the C ABI; returns the fields of its JSON line."""
    import torch
    from paper_2006_12575_b200 import binding as B
    from paper_2006_12575_b200 import synth
    cfg = UNET_CFGS[cfg_id]
    args = argparse.Namespace(cfg=cfg_id, workload=workload, steps=steps, warmup=warmup, sw_batch=sw_batch,
                              no_graph=not graph, se_ratio=se_ratio)
    peaks = measured_peaks()
    D, H, W = cfg["vol"]
    V = D * H * W
    # se_ratio > 0: the SEU-Net variant (every level's conv stack ends in a squeeze-and-excitation residual step)
    net = B.lamp_unet_create(B.unet_spec(cfg["levels"], cfg["ch"], cfg["cpl"], 1, cfg["K"], se_ratio=args.se_ratio))
    nl = B.lamp_unet_num_layers(net)
    g = torch.Generator().manual_seed(10 * args.cfg + 1)
    wflat = torch.zeros(B.lamp_unet_weight_count(net), dtype=torch.float32)
    for i in range(nl):
        wo, bo, d = B.lamp_unet_param_layout(net, i)
        taps = d.ksize ** 3
        fan = (1 if d.transposed else taps) * d.c_in
        n = taps * d.c_in * d.c_out
        wflat[wo:wo + n] = torch.randn(n, generator=g) * (2.0 / fan) ** 0.5
    wd = wflat.cuda().to(torch.bfloat16)
    bflat = torch.zeros(B.lamp_unet_bias_count(net), dtype=torch.float32)
    for i in range(nl):
        so, cr = B.lamp_unet_se_layout(net, i)
        if cr:                                   # squeeze-and-excitation parameters: small random values
            c = B.lamp_unet_param_layout(net, i)[2].c_out
            bflat[so:so + 2 * c * cr + c + cr] = torch.randn(2 * c * cr + c + cr, generator=g) * 0.3
    bd = bflat.cuda()
    key = (args.cfg, D, H, W)
    if key not in _VOLUMES:                      # the 512 x 512 x 128 volume takes 15 s to draw: once per process
        _VOLUMES[key] = synth.ct_volume((D, H, W), 40) if args.cfg == 4 else synth.blurred_noise((D, H, W), 2.0, 10 * args.cfg)
    vol = _VOLUMES[key]
    hx = torch.from_numpy(vol).to(torch.bfloat16).reshape(1, D, H, W, 1).pin_memory()
    x = hx.cuda()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    out = dict(n_gpus=1, steps=args.steps, warmup=args.warmup, higher_is_better=True, scaling="weak", vs_baseline=None,
               dtype="bf16", data="synthetic", unit="voxels/s")
    if args.se_ratio:
        out["variant"] = f"SEU-Net, reduction ratio {args.se_ratio} (the roofline floor below is the plain network's)"
    if args.workload == "unet_train":
        lab = torch.from_numpy(synth.labels_quartiles((D, H, W), 10 * args.cfg + 2, cfg["K"], 4.0)).reshape(-1).cuda()
        loss = torch.zeros(1, dtype=torch.float32, device="cuda")
        gw = torch.empty(B.lamp_unet_weight_count(net), dtype=torch.float32, device="cuda")
        gb = torch.empty(B.lamp_unet_bias_count(net), dtype=torch.float32, device="cuda")
        nbytes = B.lamp_unet_workspace_bytes(net, 1, D, H, W, B.MODE_TRAIN)
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        fn = lambda: B.lamp_unet_train_step(net, wd, bd, x, lab, loss, gw, gb, None, ws)
        flops = 3 * unet_fwd_flops(cfg)
        floor_ms = unet_floor_ms(cfg, True, peaks)
        out.update(metric="unet_train_step_voxels_per_s", config=dict(workload=f"configs[{args.cfg}] U-Net forward+backward",
                                                                         workspace_bytes=nbytes))
    elif args.workload == "unet_infer":
        # the output of both inference modes is the segmentation (arg-max) map; the sliding window writes no
        # probabilities either
        seg = torch.empty(V, dtype=torch.uint8, device="cuda")
        nbytes = B.lamp_unet_workspace_bytes(net, 1, D, H, W, B.MODE_INFER)
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        fn = lambda: B.lamp_unet_forward(net, wd, bd, x, None, seg, ws)
        flops = unet_fwd_flops(cfg)
        floor_ms = unet_floor_ms(cfg, False, peaks, probs_out=False)
        out.update(metric="unet_whole_volume_infer_voxels_per_s",
                   config=dict(workload=f"configs[{args.cfg}] whole-volume forward, output: arg-max map", workspace_bytes=nbytes))
    else:
        patch = (64, 64, 64)
        seg = torch.empty(V, dtype=torch.uint8, device="cuda")
        nbytes = B.lamp_sliding_window_workspace_bytes(net, D, H, W, patch, 0.25, args.sw_batch)
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        fn = lambda: B.lamp_sliding_window_infer(net, wd, bd, x, patch, 0.25, args.sw_batch, 1, None, seg, ws)
        pc = dict(cfg, vol=patch)
        npatch = 1
        for n_, p_ in zip((D, H, W), patch):
            s_ = 48
            k = (n_ - p_) // s_ + 1
            npatch *= k + (1 if (k - 1) * s_ != n_ - p_ else 0)
        flops = npatch * unet_fwd_flops(pc)
        # every patch's forward pass, then the blend: patch probabilities written and read once (fp32), one label out
        floor_ms = npatch * unet_floor_ms(cfg, False, peaks, vol=patch) + \
            (npatch * 64 ** 3 * 8.0 * cfg["K"] + V) / (peaks["hbm_gbs"] * 1e9) * 1e3
        out.update(metric="unet_sliding_window_infer_voxels_per_s",
                   config=dict(workload=f"configs[{args.cfg}] sliding window 64^3, overlap 0.25, gaussian", patches=npatch,
                               sw_batch=args.sw_batch, workspace_bytes=nbytes))
    for _ in range(args.warmup):
        fn()
    torch.cuda.synchronize()
    t0, t1 = ev(), ev()
    t0.record()
    for _ in range(args.steps):
        fn()
    t1.record()
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / args.steps
    if B.lamp_get_async_status() != 0:
        raise SystemExit("device status not ok")
    out.update(value=round(V / (ms * 1e-3), 1), ms_per_step=round(ms, 3), tflops=round(flops / (ms * 1e-3) / 1e12, 2),
               seconds_per_volume=round(ms * 1e-3, 5))
    out["roofline"] = dict(bound="sum over the steps of max(tensor, hbm)", floor_ms=round(floor_ms, 3),
                           frac=round(floor_ms / ms, 3), peak_source=peaks["source"],
                           peaks=dict(bf16_tflops=peaks["bf16"], hbm_gbs=peaks["hbm_gbs"]))
    if args.no_graph:
        B.lamp_unet_destroy(net)
        return out
    # the same call captured once in a CUDA graph and replayed: what the launch-bound deep levels cost in host launches
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                fn()
            for _ in range(max(1, args.warmup)):
                g.replay()
            side.synchronize()
            t0, t1 = ev(), ev()
            t0.record()
            for _ in range(args.steps):
                g.replay()
            t1.record()
            side.synchronize()
        gms = t0.elapsed_time(t1) / args.steps
        if B.lamp_get_async_status() != 0:
            raise SystemExit("device status not ok")
        out["graph_replay"] = dict(ms_per_step=round(gms, 3), value=round(V / (gms * 1e-3), 1))
    except RuntimeError as e:
        out["graph_replay"] = dict(error=str(e)[:120])
    B.lamp_unet_destroy(net)
    return out


def run_unet(args):
    import torch
    from paper_2006_12575_b200 import build as lamp_build
    lamp_build.build()
    torch.cuda.set_device(0)
    print(json.dumps(measure_unet(args.workload, args.cfg, args.steps, args.warmup, args.sw_batch, not args.no_graph,
                                  args.se_ratio)), flush=True)


def run_unet_dp(args):
    """Data-parallel training: every rank runs the U-Net training step on its own volume, the flat fp32 gradients
    are averaged over the ranks (bucketed all-reduce of the process group), and RMSProp updates the fp32 master copy
    and the bf16 copy the convolutions read.  One JSON line from rank 0: voxels of all ranks over the slowest rank."""
    import torch
    import torch.distributed as dist
    from paper_2006_12575_b200 import binding as B
    from paper_2006_12575_b200 import build as lamp_build
    from paper_2006_12575_b200 import replicas, synth
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        lamp_build.build()
    if world > 1:
        dist.barrier()
    cfg = UNET_CFGS[args.cfg]
    D, H, W = cfg["vol"]
    V = D * H * W
    net = B.lamp_unet_create(B.unet_spec(cfg["levels"], cfg["ch"], cfg["cpl"], 1, cfg["K"]))
    g = torch.Generator().manual_seed(10 * args.cfg + 1)              # the same initial weights on every rank
    master = torch.zeros(B.lamp_unet_weight_count(net), dtype=torch.float32)
    for i in range(B.lamp_unet_num_layers(net)):
        wo, bo, d = B.lamp_unet_param_layout(net, i)
        taps = d.ksize ** 3
        n = taps * d.c_in * d.c_out
        master[wo:wo + n] = torch.randn(n, generator=g) * (2.0 / ((1 if d.transposed else taps) * d.c_in)) ** 0.5
    master = master.to(dev)
    wd = master.to(torch.bfloat16)
    bmaster = torch.zeros(B.lamp_unet_bias_count(net), dtype=torch.float32, device=dev)
    vw, vb = torch.zeros_like(master), torch.zeros_like(bmaster)
    x = torch.from_numpy(synth.blurred_noise((D, H, W), 2.0, 10 * args.cfg + 100 * rank)).to(torch.bfloat16).reshape(1, D, H, W, 1).to(dev)
    lab = torch.from_numpy(synth.labels_quartiles((D, H, W), 10 * args.cfg + 2 + 100 * rank, cfg["K"], 4.0)).reshape(-1).to(dev)
    loss = torch.zeros(1, dtype=torch.float32, device=dev)
    gw, gb = torch.empty_like(master), torch.empty_like(bmaster)
    ws = torch.empty(B.lamp_unet_workspace_bytes(net, 1, D, H, W, B.MODE_TRAIN), dtype=torch.uint8, device=dev)

    # gradient buckets of about 32 MB that end on layer boundaries; each one's all-reduce starts on its own stream as
    # soon as the backward pass has finished it
    offs = [B.lamp_unet_param_layout(net, i)[0] for i in range(B.lamp_unet_num_layers(net))]
    starts = replicas.plan_buckets(offs, gw.numel(), 8 << 20)
    events = [torch.cuda.Event() for _ in starts]
    comm = torch.cuda.Stream()

    def step():
        replicas.train_step_overlapped(B, net, wd, bmaster, x, lab, loss, gw, gb, None, ws, starts, events, comm)
        B.lamp_rmsprop_step(gw, master, vw, wd)
        B.lamp_rmsprop_step(gb, bmaster, vb, None)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    losses = []
    for _ in range(args.warmup):
        step()
        losses.append(float(loss.item()))
    sync_all()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        step()
    t1.record()
    sync_all()
    losses.append(float(loss.item()))
    ms = replicas.job_time_ms(t0.elapsed_time(t1), dev) / args.steps
    status = B.lamp_get_async_status()
    if rank == 0:
        if status != 0:
            raise SystemExit("device status not ok")
        out = dict(metric="unet_data_parallel_train_voxels_per_s", value=round(world * V / (ms * 1e-3), 1), unit="voxels/s",
                   n_gpus=world, steps=args.steps, warmup=args.warmup, ms_per_step=round(ms, 3), higher_is_better=True,
                   scaling="weak", vs_baseline=None, dtype="bf16", data="synthetic",
                   config=dict(workload=f"configs[{args.cfg}] U-Net training step + gradient average over {world} replica(s) "
                                        "+ RMSProp update", gradient_bytes=int(gw.numel() + gb.numel()) * 4,
                               exchange=f"{len(starts)} buckets, each all-reduced on a second stream as soon as the backward pass "
                                        "has finished it"),
                   loss_first_last=[round(losses[0], 5), round(losses[-1], 5)] if losses else None)
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_sliding_dp(args):
    """Sliding-window inference of one volume with the patches split over the replicas (one reduction of the class
    sums and weight totals).  One JSON line from rank 0: voxels of the volume over the slowest rank's time."""
    import torch
    import torch.distributed as dist
    from paper_2006_12575_b200 import binding as B
    from paper_2006_12575_b200 import build as lamp_build
    from paper_2006_12575_b200 import replicas, synth
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        lamp_build.build()
    if world > 1:
        dist.barrier()
    cfg = UNET_CFGS[args.cfg]
    D, H, W = cfg["vol"]
    K = cfg["K"]
    patch = (64, 64, 64)
    net = B.lamp_unet_create(B.unet_spec(cfg["levels"], cfg["ch"], cfg["cpl"], 1, K))
    g = torch.Generator().manual_seed(10 * args.cfg + 1)
    wflat = torch.zeros(B.lamp_unet_weight_count(net), dtype=torch.float32)
    for i in range(B.lamp_unet_num_layers(net)):
        wo, bo, d = B.lamp_unet_param_layout(net, i)
        taps = d.ksize ** 3
        n = taps * d.c_in * d.c_out
        wflat[wo:wo + n] = torch.randn(n, generator=g) * (2.0 / ((1 if d.transposed else taps) * d.c_in)) ** 0.5
    wd = wflat.to(dev).to(torch.bfloat16)
    bd = torch.zeros(B.lamp_unet_bias_count(net), dtype=torch.float32, device=dev)
    vol = synth.ct_volume((D, H, W), 40) if args.cfg == 4 else synth.blurred_noise((D, H, W), 2.0, 10 * args.cfg)
    x = torch.from_numpy(vol).to(torch.bfloat16).reshape(1, D, H, W, 1).to(dev)
    sums = torch.empty((K, D, H, W), dtype=torch.float32, device=dev)
    wsum = torch.empty((D, H, W), dtype=torch.float32, device=dev)
    seg = torch.empty(D * H * W, dtype=torch.uint8, device=dev)
    ws = torch.empty(B.lamp_sliding_window_workspace_bytes(net, D, H, W, patch, 0.25, args.sw_batch), dtype=torch.uint8, device=dev)
    fn = lambda: replicas.sliding_window_sharded(B, net, wd, bd, x, patch, 0.25, args.sw_batch, 1, sums, wsum, seg, ws)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        fn()
    sync_all()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        fn()
    t1.record()
    sync_all()
    ms = replicas.job_time_ms(t0.elapsed_time(t1), dev) / args.steps
    status = B.lamp_get_async_status()
    if rank == 0:
        if status != 0:
            raise SystemExit("device status not ok")
        print(json.dumps(dict(metric="unet_sliding_window_sharded_voxels_per_s", value=round(D * H * W / (ms * 1e-3), 1),
                              unit="voxels/s", n_gpus=world, steps=args.steps, warmup=args.warmup, ms_per_step=round(ms, 3),
                              seconds_per_volume=round(ms * 1e-3, 5), higher_is_better=True, scaling="strong", vs_baseline=None,
                              dtype="bf16", data="synthetic",
                              config=dict(workload=f"configs[{args.cfg}] sliding window 64^3, overlap 0.25, gaussian; patches split "
                                                   f"over {world} replica(s), class sums and weight totals all-reduced",
                                          patches=B.lamp_sliding_window_num_patches(D, H, W, patch, 0.25),
                                          sw_batch=args.sw_batch, reduced_bytes=int(sums.numel() + wsum.numel()) * 4))), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_hbm(args):
    """HBM-bound kernels of the path on their own, through the C ABI: achieved GB/s of algorithmic bytes
    against the measured copy bandwidth."""
    import torch
    from paper_2006_12575_b200 import binding as B
    from paper_2006_12575_b200 import build as lamp_build
    lamp_build.build()
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timed(fn, flush):
        for _ in range(args.warmup):
            fn()
        tot = 0.0
        for _ in range(args.steps):
            flush.add_(1)                                # > L2: evicts the previous iteration's lines
            a, b = ev(), ev()
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            tot += a.elapsed_time(b)
        return tot / args.steps

    flush = torch.zeros(256 << 20, dtype=torch.uint8, device="cuda")
    res = {}
    D = H = W = 128
    for C in (32, 64):
        shape = (1, D, H, W, C)
        y = torch.randn(shape, device="cuda").to(torch.bfloat16)
        dz = torch.randn(shape, device="cuda").to(torch.bfloat16)
        z = torch.empty_like(y)
        dy = torch.empty_like(y)
        yf = y.float()
        stats = torch.stack([yf.sum(dim=(1, 2, 3)), (yf * yf).sum(dim=(1, 2, 3))], dim=-1).double().contiguous()
        mr = torch.empty((1, C, 2), dtype=torch.float32, device="cuda")
        sums = torch.empty((1, C, 2), dtype=torch.float64, device="cuda")
        n = y.numel()
        ms = timed(lambda: B.lamp_instnorm_relu_fwd(y, stats, 1e-5, mr, z), flush)
        res[f"instnorm_relu_fwd C={C}"] = dict(ms=round(ms, 4), bytes=4 * n, gbs=round(4 * n / ms / 1e6, 1))
        ms = timed(lambda: B.lamp_instnorm_relu_bwd(dz, None, y, mr, sums, dy), flush)
        res[f"instnorm_relu_bwd C={C}"] = dict(ms=round(ms, 4), bytes=10 * n, gbs=round(10 * n / ms / 1e6, 1))
        del y, dz, z, dy, yf
    # convolutions of the network whose FLOPs per byte sit below the machine balance: the one-channel first layer,
    # the 2x2x2 transposed (up) conv into a concat slice and the stride-2 (down) conv at the top level
    x1 = torch.randn((1, D, H, W, 1), device="cuda").to(torch.bfloat16)
    for C in (32, 64):
        w1 = (torch.randn((27, C, 1), device="cuda") * 0.2).to(torch.bfloat16)
        b1 = torch.zeros(C, device="cuda")
        y1 = torch.empty((1, D, H, W, C), dtype=torch.bfloat16, device="cuda")
        st1 = torch.zeros((1, C, 2), dtype=torch.float64, device="cuda")
        desc = B.conv_desc(1, C, 3, 1, 1, False)
        nb = x1.numel() * 2 + y1.numel() * 2
        ms = timed(lambda: B.lamp_conv3d_fwd(desc, x1, w1, b1, y1, st1), flush)
        res[f"first-layer conv 1->{C}"] = dict(ms=round(ms, 4), bytes=nb, gbs=round(nb / ms / 1e6, 1))
        del y1
    xu = torch.randn((1, D // 2, H // 2, W // 2, 64), device="cuda").to(torch.bfloat16)
    wu = (torch.randn((8, 32, 64), device="cuda") * 0.1).to(torch.bfloat16)
    cat = torch.zeros((1, D, H, W, 64), dtype=torch.bfloat16, device="cuda")
    desc = B.conv_desc(64, 32, 2, 2, 0, True)
    nb = xu.numel() * 2 + cat.numel()                    # the written slice is half of the concat buffer
    ms = timed(lambda: B.lamp_conv3d_fwd(desc, xu, wu, torch.zeros(32, device="cuda"), B.tensor(cat, 32, 32)), flush)
    res["up conv 64->32 into concat slice"] = dict(ms=round(ms, 4), bytes=nb, gbs=round(nb / ms / 1e6, 1))
    xd = torch.randn((1, D, H, W, 32), device="cuda").to(torch.bfloat16)
    wd = (torch.randn((27, 64, 32), device="cuda") * 0.05).to(torch.bfloat16)
    yd = torch.empty((1, D // 2, H // 2, W // 2, 64), dtype=torch.bfloat16, device="cuda")
    std = torch.zeros((1, 64, 2), dtype=torch.float64, device="cuda")
    desc = B.conv_desc(32, 64, 3, 2, 1, False)
    nb = xd.numel() * 2 + yd.numel() * 2
    ms = timed(lambda: B.lamp_conv3d_fwd(desc, xd, wd, torch.zeros(64, device="cuda"), yd, std), flush)
    res["down conv 32->64 stride 2"] = dict(ms=round(ms, 4), bytes=nb, gbs=round(nb / ms / 1e6, 1))
    del xu, cat, xd, yd
    # parameter update over a flat buffer the size of the 175 M-parameter network's weights
    npar = 175 * 1000 * 1000
    gq = torch.randn(npar, device="cuda")
    wq = torch.randn(npar, device="cuda")
    vq = torch.rand(npar, device="cuda")
    wq16 = torch.empty(npar, dtype=torch.bfloat16, device="cuda")
    ms = timed(lambda: B.lamp_rmsprop_step(gq, wq, vq, wq16, 1e-3, 0.99, 1e-8), flush)
    res["rmsprop step 175 M parameters"] = dict(ms=round(ms, 4), bytes=22 * npar, gbs=round(22 * npar / ms / 1e6, 1))
    del gq, wq, vq, wq16
    # overlap-add on the 512 x 512 x 128 volume: 363 patches of 64^3, K = 10
    K, P = 10, (64, 64, 64)
    Dv, Hv, Wv = 512, 512, 128
    pp = torch.rand((363, 64 ** 3, K), device="cuda")
    planar = torch.empty((K, Dv, Hv, Wv), dtype=torch.float32, device="cuda")
    seg = torch.empty(Dv * Hv * Wv, dtype=torch.uint8, device="cuda")
    nbytes = pp.numel() * 4 + planar.numel() * 4 + seg.numel()
    ms = timed(lambda: B.lamp_overlap_add(pp, K, Dv, Hv, Wv, P, 0.25, 1, planar, seg), flush)
    res["overlap_add 512x512x128"] = dict(ms=round(ms, 4), bytes=nbytes, gbs=round(nbytes / ms / 1e6, 1))
    for v in res.values():
        v["frac_of_measured_copy"] = round(v["gbs"] / peaks["hbm_gbs"], 3)
    print(json.dumps(dict(metric="hbm_bound_kernels_gbs", unit="GB/s", peak=peaks["hbm_gbs"], peak_source=peaks["source"],
                          l2="a 256 MiB buffer is rewritten between timed calls", steps=args.steps, warmup=args.warmup,
                          kernels=res)), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="lamp", choices=["lamp", "reference"])
    ap.add_argument("--channels", default=",".join(str(c) for c in CHANNELS))
    ap.add_argument("--workload", default="conv_sweep", choices=["conv_sweep", "unet_train", "unet_infer", "sliding", "hbm", "unet_train_dp", "sliding_dp"])
    ap.add_argument("--cfg", type=int, default=2)
    ap.add_argument("--sw-batch", type=int, default=32)
    ap.add_argument("--no-graph", action="store_true", help="U-Net workloads: skip the CUDA-graph replay timing")
    ap.add_argument("--se-ratio", type=int, default=0, help="U-Net workloads: SEU-Net variant with this reduction ratio (0: plain)")
    ap.add_argument("--no-unet", action="store_true", help="conv sweep: leave out the U-Net workloads that follow it")
    args = ap.parse_args()
    if args.workload == "hbm":
        run_hbm(args)
        return
    if args.workload == "unet_train_dp":
        run_unet_dp(args)
        return
    if args.workload == "sliding_dp":
        run_sliding_dp(args)
        return
    if args.workload != "conv_sweep":
        run_unet(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
