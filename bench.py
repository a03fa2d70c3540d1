#!/usr/bin/env python
"""Benchmark of the parallel autoregressive sampler on B200.

One step = one ``jacobi_sample`` call (the whole hot path: every Jacobi
iteration's masked forward pass, the fused sampling and compare, the device-side
loop) over one batch of the seeded synthetic workload.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--mode jacobi|gs_jacobi|jacobi_gs]
    python bench.py --impl reference ...      # the CPU oracle on a bounded sample of the same workload
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

import synth_inputs as si  # noqa: E402

METRIC = "jacobi_ar_samples_per_sec"
UNIT = "samples/s"
DEFAULT_WORKLOAD = "made_4096"


# ------------------------------------------------------------------ workload
def conv_live_macs_per_image(cfg) -> int:
    """Unmasked multiply-accumulates of one forward pass of the masked-conv stack for one image
    (four full taps and the colour-group-masked centre tap per 3x3 layer, masked 1x1 head)."""
    ch, n_in = cfg.ch, cfg.in_ch
    grp = (n_in * np.arange(ch)) // ch
    per_pixel = 0
    for l in range(cfg.layers):
        cin = n_in if l == 0 else ch
        gi = np.arange(n_in) if l == 0 else grp
        centre = (gi[None, :] < grp[:, None]) if l == 0 else (gi[None, :] <= grp[:, None])
        per_pixel += 4 * cin * ch + int(centre.sum())
    head = grp[None, :] <= (np.arange(n_in * cfg.C) // cfg.C)[:, None]
    per_pixel += int(head.sum())
    return per_pixel * cfg.height * cfg.width


def live_macs_per_sample(cfg) -> int:
    """Unmasked multiply-accumulates of one forward pass for one sample."""
    if cfg.kind == "conv":
        return conv_live_macs_per_image(cfg)
    D, C = cfg.D, cfg.C
    deg = [np.arange(1, D + 1)]
    for h in cfg.H:
        deg.append(1 + (np.arange(h) * (D - 1)) // h)
    deg.append(np.repeat(np.arange(1, D + 1), C))
    total = 0
    for l in range(len(cfg.H) + 1):
        srt = np.sort(deg[l])
        side = "left" if l == len(cfg.H) else "right"      # outputs read strictly smaller degrees
        total += int(np.searchsorted(srt, deg[l + 1], side=side).sum())
    return total


def dense_macs_per_sample(cfg) -> int:
    w = [cfg.D, *cfg.H, cfg.D * cfg.C]
    return int(sum(w[i] * w[i + 1] for i in range(len(w) - 1)))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def algorithmic_bytes_per_pass(cfg) -> float:
    """Bytes one forward pass has to move at least: live weights once, noise, symbols in and out."""
    live = live_macs_per_sample(cfg)
    if cfg.kind == "conv":
        live = live // (cfg.height * cfg.width)      # a conv weight serves every pixel
    noise = cfg.batch * cfg.D * (cfg.C if cfg.noise_kind == si.NOISE_GUMBEL else 1) * 4
    return 2.0 * live + noise + 2.0 * cfg.batch * cfg.D


def recorded_traffic(workload: str):
    """DRAM bytes per launch from the committed ncu record, or None once the kernels have changed."""
    import glob
    import hashlib
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    rec = dict(l.split() for l in open(path) if l.strip() and not l.startswith("#"))
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2002_03629_b200", "csrc")
    for f in sorted(glob.glob(csrc + "/*.cu") + glob.glob(csrc + "/*.cuh") + glob.glob(csrc + "/*.h")):
        h.update(open(f, "rb").read())
    if h.hexdigest()[:16] != rec.get("csrc_sha") or workload not in rec:
        return None
    return int(rec[workload])


class ClockSampler:
    """nvidia-smi clock and throttle-reason samples during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(gpu_index)], stdout=self.f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.flush()
        rows = [r.strip().split(", ") for r in open(self.f.name) if r.strip()]
        os.unlink(self.f.name)
        sm, reasons, mx = [], set(), None
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1]))
                mx = float(r[2])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.strip().lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out["sm_mhz"] = float(np.median(sm))
            out["sm_max_mhz"] = mx
        out["reasons"] = sorted(reasons)
        out["samples"] = len(sm)
        return out


MODES = {"jacobi": 0, "gauss_seidel": 1, "gs_jacobi": 2, "jacobi_gs": 3}


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of per-rank timings (no-op without a process group).  Replicas exchange
    nothing else: each rank samples its own batch."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_rate(samples_per_rank: int, steps: int, world: int, seconds: float) -> float:
    """Samples per second of all replicas together, against the slowest rank's time."""
    return samples_per_rank * steps * world / seconds


def make_inputs(cfg):
    if cfg.kind == "conv":
        W, b = si.conv_weights(cfg)
        return W, b, si.conv_lut(cfg), si.draw_noise(cfg)
    W, b = si.made_weights(cfg)
    return W, b, si.made_lut(cfg), si.draw_noise(cfg)


# -------------------------------------------------------------- reference arm
def oracle_sample_time(cfg, W, b, lut, noise, mode, block, n_samples, threads):
    """Oracle wall time for n_samples of the workload in the given mode (as it stands, untuned)."""
    import oracle
    orc = oracle.from_config(cfg, W, b, lut)
    nk = cfg.noise_kind

    def one(i):
        if mode == "jacobi":
            return orc.jacobi(noise[i], nk)[1]
        if mode == "gs_jacobi":
            return orc.gs_jacobi(noise[i], nk, block)[1]
        if mode == "jacobi_gs":
            return orc.jacobi_gs(noise[i], nk, block)[1]
        orc.gauss_seidel(noise[i], nk)
        return 1
    t0 = time.perf_counter()
    its = orc.map_batch(one, n_samples, threads)
    dt = time.perf_counter() - t0
    return dt, its


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    W, b, lut, noise = make_inputs(cfg)
    cores = os.cpu_count() or 1
    n = min(cfg.batch, max(1, args.ref_samples))
    for _ in range(args.warmup and 1):
        oracle_sample_time(cfg, W, b, lut, noise, args.mode, args.block, min(n, cores), cores)
    total, its = 0.0, []
    for _ in range(args.steps):
        dt, it = oracle_sample_time(cfg, W, b, lut, noise, args.mode, args.block, n, cores)
        total += dt
        its += it
    value = n * args.steps / total
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "mode": args.mode, "block": args.block, "batch": cfg.batch,
                       "sample": f"{n} of {cfg.batch} samples per step"},
            "iters_per_sample_mean": float(np.mean(its)),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(cores, n), "kind": "oracle",
                             "sample": f"{n} samples x {args.steps} steps, {args.mode}"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# -------------------------------------------------------------------- our arm
def run_ours(args, cfg):
    import torch
    import torch.distributed as dist

    import __graft_entry__ as ge
    ge.build()
    import paper_2002_03629_b200 as pkg

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    W, b, lut, noise = make_inputs(cfg)
    model = pkg.Model.from_config(cfg, W, b, lut)
    del W, b
    nk, mode, block = cfg.noise_kind, MODES[args.mode], args.block
    h_noise = torch.from_numpy(noise).pin_memory()
    d_noise = h_noise.cuda()
    out = torch.empty((cfg.batch, cfg.D), dtype=torch.uint8, device="cuda")
    iters = torch.empty((cfg.batch,), dtype=torch.int32, device="cuda")
    h_out = torch.empty((cfg.batch, cfg.D), dtype=torch.uint8).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # larger than the 126 MB L2

    def step():
        return pkg.jacobi_sample(model, d_noise, nk, None, mode, block, 0, out, iters)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        rc = step()
        if rc != 0:
            raise RuntimeError(f"jacobi_sample returned {rc}")
    it_np = iters.cpu().numpy()
    stats = model.stats()

    # ---- device-resident timing: K steps, L2 flushed between them, CUDA events per step
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for s, e in ev:
        flush.zero_()
        s.record()
        step()
        e.record()
    barrier()
    ms = [s.elapsed_time(e) for s, e in ev]
    total_ms = float(sum(ms))
    if sampler and not args.profile:
        # the timed region is milliseconds long: keep the same load running (untimed) until
        # nvidia-smi has had time to take a few samples of the clocks under it
        t_end = time.perf_counter() + 0.8
        while time.perf_counter() < t_end:
            step()
    clocks = sampler.stop() if sampler else None

    # ---- end to end: the host-buffer call of the C ABI, pinned host noise in, host samples out; the
    # upload, the solve and the download are all inside the call and inside the timed region
    pkg.jacobi_sample_host(model, h_noise, nk, None, mode, block, 0, h_out)       # allocates the staging buffers
    if not torch.equal(h_out, out.cpu()):
        raise RuntimeError("jacobi_sample_host and jacobi_sample disagree")
    barrier()
    t_e2e = []
    for _ in range(1 if args.profile else args.steps):
        flush.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        pkg.jacobi_sample_host(model, h_noise, nk, None, mode, block, 0, h_out)
        t_e2e.append(time.perf_counter() - t0)
    e2e_s = float(sum(t_e2e)) * (args.steps / len(t_e2e))

    # ---- the same kernels in strict sequential order (speedup denominators)
    seq = {}
    if args.seq and rank == 0 and not args.profile:
        for name, opt in (("seq_skip", 1), ("seq_full", 0)):
            if name == "seq_full" and args.seq == "skip":
                continue
            model.set_option(pkg.JS_OPT_SEQ_SKIP, opt)
            out2 = torch.empty_like(out)
            pkg.sequential_sample(model, d_noise, nk, out2)       # warm-up
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            flush.zero_()
            s.record()
            pkg.sequential_sample(model, d_noise, nk, out2)
            e.record()
            torch.cuda.synchronize()
            seq[name + "_ms"] = s.elapsed_time(e)
            seq[name + "_matches_jacobi"] = bool(torch.equal(out2, out))
        model.set_option(pkg.JS_OPT_SEQ_SKIP, 0)

    total_ms, e2e_s = max_over_ranks([total_ms, e2e_s], device="cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    n_samples = cfg.batch * args.steps * world
    value = whole_job_rate(cfg.batch, args.steps, world, total_ms / 1e3)
    live = live_macs_per_sample(cfg)
    flops_per_launch = 2.0 * live * cfg.batch * stats.iterations
    ms_launch = total_ms / args.steps
    bytes_per_launch = algorithmic_bytes_per_pass(cfg) * stats.iterations
    dtype = "bf16" if cfg.prec == si.PREC_BF16 else "f32"
    kernel_name = "conv_tc_kernel" if cfg.kind == "conv" else ("made_tc_kernel" if stats.path == 0 else "made_generic_kernel")
    # bound of the dominant kernel: by arithmetic intensity against the ridge of the measured peaks
    ridge = peaks["bf16_tflops"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    if flops_per_launch / bytes_per_launch >= ridge:
        achieved = flops_per_launch / (ms_launch / 1e3) / 1e12
        peak = peaks["bf16_tflops"]
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "peak_source": peaks["source"] + " burst bf16 (kernel timed alone)",
                    "note": "live (unmasked) MACs x 2 x batch x forward passes executed"}
    else:
        achieved = bytes_per_launch / (ms_launch / 1e3) / 1e9
        peak = peaks["hbm_gbs"]
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "peak_source": peaks["source"] + " copy bandwidth",
                    "note": "(live weights + noise + symbols) x forward passes executed; skipped tiles are not subtracted"}
    roofline.update({"traffic": recorded_traffic(cfg.name), "kernel": kernel_name + " (one launch = all iterations of one call)",
                     "flops_per_launch": flops_per_launch, "bytes_per_launch": bytes_per_launch,
                     "ms_per_launch": ms_launch})

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_launch, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": dtype, "data": "synthetic",
            "config": {"workload": cfg.name, "mode": args.mode, "block": block, "batch": cfg.batch, "T": cfg.D,
                       "C": cfg.C, "hidden": list(cfg.H) if cfg.kind == "made" else [cfg.ch] * cfg.layers,
                       "parallelism": f"replicas x{world}",
                       "l2": "256 MB written between timed steps (L2 flush)"},
            "iters_per_sample": {"mean": float(it_np.mean()), "max": int(it_np.max()),
                                 "forward_passes": int(stats.iterations)},
            "kernel_path": "tensor-core" if stats.path == 0 else "cuda-core",
            "tiles": {"issued": int(stats.tiles_issued), "skipped": int(stats.tiles_skipped)},
            "roofline": roofline,
            "e2e": {"value": n_samples / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(h_noise.numel() * 4),
                    "d2h_bytes_per_step": int(h_out.numel())},
            "gpu_launches": args.steps,
            "clocks": clocks}
    if seq:
        line["sequential_on_gpu"] = seq
        for k in ("seq_skip_ms", "seq_full_ms"):
            if k in seq:
                line["speedup_vs_" + k[:-3]] = seq[k] / ms_launch

    # ---- CPU baseline: the oracle on a bounded sample of the same workload
    if not args.no_cpu_baseline and not args.profile:
        import oracle
        oracle.build()
        W, b, lut, noise2 = make_inputs(cfg)
        cores = os.cpu_count() or 1
        n = min(cfg.batch, args.ref_samples)
        dt, its = oracle_sample_time(cfg, W, b, lut, noise2, args.mode, block, n, cores)
        line["cpu_baseline"] = {"value": n / dt, "unit": UNIT, "cores": min(cores, n), "kind": "oracle",
                                "sample": f"{n} of {cfg.batch} samples, {args.mode}, {dt:.1f} s",
                                "iters_per_sample_mean": float(np.mean(its))}
        line["iters_per_sample"]["oracle_mean_on_sample"] = float(np.mean(its))
        line["iters_per_sample"]["gpu_mean_on_same_samples"] = float(it_np[:n].mean())
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=[k for k, v in si.CONFIGS.items()])
    ap.add_argument("--mode", default="jacobi", choices=list(MODES))
    ap.add_argument("--block", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (debugging)")
    ap.add_argument("--seq", default="skip", choices=["", "skip", "full"],
                    help="also time the strict sequential order: banded only, or banded and full")
    ap.add_argument("--ref-samples", type=int, default=0,
                    help="samples per step of the CPU oracle (0: sized for roughly 15 s of CPU work)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile", action="store_true",
                    help="only the warm-up and the timed steps (for short runs under a profiler)")
    args = ap.parse_args()
    cfg = si.CONFIGS[args.workload]
    if args.batch:
        cfg = si.scaled(cfg, batch=args.batch)
    if args.mode in ("gs_jacobi", "jacobi_gs") and args.block <= 0:
        args.block = cfg.blocks[0] if cfg.blocks else 64
    if args.ref_samples <= 0:
        cores = os.cpu_count() or 1
        per_sample_s = 4.0 * live_macs_per_sample(cfg) / 0.6e9          # a few forward passes at ~0.6 GMAC/s
        args.ref_samples = int(min(cfg.batch, max(cores, 15.0 * cores / per_sample_s)))
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
