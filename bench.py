#!/usr/bin/env python
"""Benchmark of the parallel autoregressive sampler on B200.

One step = one ``jacobi_sample`` call (the whole hot path: every Jacobi
iteration's masked forward pass, the fused sampling and compare, the device-side
loop) over one batch of the seeded synthetic workload.  Prints ONE JSON line: the
headline workload (``--workload``, default the largest masked MLP) on top, and under
``workloads`` every seeded config measured the same way in the same run.

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


def config_of(cfg, mode, block, world):
    """The `config` object of the JSON line: the same in both arms, so that the two lines can be paired."""
    return {"workload": cfg.name, "mode": mode, "block": block, "batch": cfg.batch, "T": cfg.D, "C": cfg.C,
            "hidden": list(cfg.H) if cfg.kind == "made" else [cfg.ch] * cfg.layers,
            "parallelism": f"replicas x{world}",
            "l2": "256 MB written between timed GPU steps (L2 flush)"}


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
            "config": config_of(cfg, args.mode, args.block, args.gpus),
            "iters_per_sample_mean": float(np.mean(its)),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(cores, n), "kind": "oracle",
                             "sample": f"{n} samples x {args.steps} steps, {args.mode}"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# -------------------------------------------------------------------- our arm
NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 7700.0}      # data-sheet figures, for context beside the measured peaks


def roofline_of(cfg, stats, it_np, ms_launch, peaks):
    """Roofline record of one call.  Algorithmic work counts only what the method needs: the live
    (unmasked) multiply-accumulates of a forward pass for every sample that was still iterating in that
    pass (the sum of the per-sample iteration counts), and for bytes the weight tiles the passes had to
    stream (counted by the kernel: each tile once per pass, tiles behind the frontier not at all) plus
    the noise and symbols of the samples still iterating."""
    live = live_macs_per_sample(cfg)
    sample_passes = int(it_np.sum())
    flops = 2.0 * live * sample_passes
    noise_per_sample = cfg.D * (cfg.C if cfg.noise_kind == si.NOISE_GUMBEL else 1) * 4
    wbytes = float(stats.weight_bytes) if stats.weight_bytes > 0 else 2.0 * live * stats.iterations
    nbytes = wbytes + (noise_per_sample + 2.0 * cfg.D) * sample_passes
    kernel_name = "conv_tc_kernel" if cfg.kind == "conv" else ("made_tc_kernel" if stats.path == 0 else "made_generic_kernel")
    ridge = peaks["bf16_tflops"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    sec = ms_launch / 1e3
    if flops / nbytes >= ridge:
        achieved, peak = flops / sec / 1e12, peaks["bf16_tflops"]
        r = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
             "peak_source": peaks["source"] + " burst bf16 (kernel timed alone)",
             "frac_of_nominal": achieved / NOMINAL["bf16_tflops"],
             "note": "2 x live (unmasked) MACs per sample x sum over samples of the passes each was still iterating in"}
    else:
        achieved, peak = nbytes / sec / 1e9, peaks["hbm_gbs"]
        r = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
             "peak_source": peaks["source"] + " copy bandwidth",
             "frac_of_nominal": achieved / NOMINAL["hbm_gbs"],
             "note": "weight tiles streamed (device-counted, once per pass, frontier-skipped tiles excluded) + noise and "
                     "symbols of the samples still iterating"}
    r.update({"traffic": recorded_traffic(cfg.name), "kernel": kernel_name + " (one launch = all iterations of one call)",
              "flops_per_launch": flops, "bytes_per_launch": nbytes, "ms_per_launch": ms_launch,
              "sample_passes": sample_passes,
              "frac_full_batch": (2.0 * live * cfg.batch * stats.iterations) / sec / 1e12 / peaks["bf16_tflops"],
              "mma_issued_tflops": float(stats.mma_flops) / sec / 1e12 if stats.mma_flops > 0 else None,
              "mma_issued_frac": float(stats.mma_flops) / sec / 1e12 / peaks["bf16_tflops"] if stats.mma_flops > 0 else None})
    return r


def measure_workload(pkg, cfg, inputs, mode_name, block, steps, warmup, world, rank, local, profile, seq, sample_clocks):
    """Times one workload on this rank.  Returns (record, extras) where extras holds what the
    headline line needs beside the record (clocks, arrays for the CPU leg)."""
    import torch
    import torch.distributed as dist

    W, b, lut, noise = inputs
    model = pkg.Model.from_config(cfg, W, b, lut)
    nk, mode = cfg.noise_kind, MODES[mode_name]
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

    for _ in range(max(warmup, 3)):
        rc = step()
        if rc != 0:
            raise RuntimeError(f"jacobi_sample returned {rc} on {cfg.name}")
    it_np = iters.cpu().numpy()
    stats = model.stats()

    # ---- device-resident timing: K steps, L2 flushed between them, CUDA events per step
    barrier()
    sampler = ClockSampler(local) if (rank == 0 and sample_clocks) else None
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for s, e in ev:
        flush.zero_()
        s.record()
        step()
        e.record()
    barrier()
    total_ms = float(sum(s.elapsed_time(e) for s, e in ev))
    if sampler and not profile:
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
    for _ in range(1 if profile else steps):
        flush.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        pkg.jacobi_sample_host(model, h_noise, nk, None, mode, block, 0, h_out)
        t_e2e.append(time.perf_counter() - t0)
    e2e_s = float(sum(t_e2e)) * (steps / len(t_e2e))

    # ---- the same model in strict sequential order (speedup denominators)
    seq_rec = {}
    if seq and rank == 0 and not profile:
        for name, opt in (("seq_cached", 2), ("seq_skip", 1), ("seq_full", 0)):
            if name == "seq_full" and seq == "skip":
                continue
            if name == "seq_cached" and not (cfg.kind == "made" and cfg.C == 1 and cfg.prec == si.PREC_BF16):
                continue          # the cached sweep serves binary bf16 masked MLPs
            model.set_option(pkg.JS_OPT_SEQ_SKIP, opt)
            out2 = torch.empty_like(out)
            pkg.sequential_sample(model, d_noise, nk, out2)       # warm-up
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            flush.zero_()
            s.record()
            pkg.sequential_sample(model, d_noise, nk, out2)
            e.record()
            torch.cuda.synchronize()
            seq_rec[name + "_ms"] = s.elapsed_time(e)
            seq_rec[name + "_us_per_position"] = 1e3 * seq_rec[name + "_ms"] / cfg.D
            seq_rec[name + "_matches_jacobi"] = bool(torch.equal(out2, out))
        model.set_option(pkg.JS_OPT_SEQ_SKIP, 2)

    total_ms, e2e_s = max_over_ranks([total_ms, e2e_s], device="cuda")
    ms_launch = total_ms / steps
    peaks = load_peaks()
    rec = {"ms_per_call": ms_launch, "samples_per_s": whole_job_rate(cfg.batch, steps, world, total_ms / 1e3),
           "mode": mode_name, "block": block, "batch": cfg.batch,
           "iters_per_sample": {"mean": float(it_np.mean()), "max": int(it_np.max()),
                                "forward_passes": int(stats.iterations)},
           "kernel_path": "tensor-core" if stats.path == 0 else "cuda-core",
           "tiles": {"issued": int(stats.tiles_issued), "skipped": int(stats.tiles_skipped)},
           "e2e": {"value": cfg.batch * steps * world / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(h_noise.numel() * 4),
                   "d2h_bytes_per_step": int(h_out.numel())}}
    if stats.path == 0:
        rec["roofline"] = roofline_of(cfg, stats, it_np, ms_launch, peaks)
    else:
        rec["roofline"] = "latency-bound (CUDA-core kernels, a few kFLOP per pass)"
    if seq_rec:
        rec["sequential_on_gpu"] = seq_rec
        for k in ("seq_cached_ms", "seq_skip_ms", "seq_full_ms"):
            if k in seq_rec:
                rec["speedup_vs_" + k[:-3]] = seq_rec[k] / ms_launch
    extras = {"clocks": clocks, "samples": out.cpu().numpy(), "iters": it_np, "steps": steps}
    model.close()
    del d_noise, flush
    torch.cuda.empty_cache()
    return rec, extras


def cpu_leg(cfg, inputs, mode_name, block, n, gpu_samples, gpu_iters):
    """The oracle, as it stands, on n samples of the workload: its rate, its iteration counts beside the
    GPU's on the same samples, and how many of those samples differ from the GPU's anywhere."""
    import oracle
    oracle.build()
    W, b, lut, noise = inputs
    cores = os.cpu_count() or 1
    orc = oracle.from_config(cfg, W, b, lut)
    nk = cfg.noise_kind

    def one(i):
        if mode_name == "jacobi":
            r = orc.jacobi(noise[i], nk)
        elif mode_name == "gs_jacobi":
            r = orc.gs_jacobi(noise[i], nk, block)
        elif mode_name == "jacobi_gs":
            r = orc.jacobi_gs(noise[i], nk, block)
        else:
            r = (orc.gauss_seidel(noise[i], nk), 1)
        return r[0], r[1]
    t0 = time.perf_counter()
    res = orc.map_batch(one, n, cores)
    dt = time.perf_counter() - t0
    its = [r[1] for r in res]
    differing = int(sum(1 for i, r in enumerate(res) if not np.array_equal(r[0], gpu_samples[i])))
    return {"value": n / dt, "unit": UNIT, "cores": min(cores, n), "kind": "oracle",
            "sample": f"{n} of {cfg.batch} samples, {mode_name}, {dt:.1f} s",
            "iters_per_sample_mean": float(np.mean(its)),
            "gpu_iters_mean_on_same_samples": float(gpu_iters[:n].mean()),
            "samples_differing_from_gpu": differing}


def measure_rnn(local: int, with_oracle: bool):
    """The recurrent-network workload (Section 5.1): gradients of a batch of sequences, the backward pass by
    back-substitution and by Jacobi_n.  Times are CUDA-event means over 20 calls after 3 warm-up calls; the
    inputs stay resident and L2 is flushed between calls."""
    import torch
    import paper_2002_03629_b200.rnn as rnn
    out = {}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for name in ("rnn_100", "rnn_100_batch"):
        cfg = si.RNN_CONFIGS[name]
        params = [torch.from_numpy(a).cuda() for a in si.rnn_weights(cfg)]
        x, r = (torch.from_numpy(a).cuda() for a in si.rnn_sequences(cfg))
        h, d, l, loss = rnn.rnn_forward(*params, x, r)
        s = torch.empty_like(l)

        def timed(fn, reps=20):
            for _ in range(3):
                fn()
            tot = 0.0
            for _ in range(reps):
                flush.fill_(1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                fn()
                b.record()
                b.synchronize()
                tot += a.elapsed_time(b)
            return tot / reps

        rec = {"batch": cfg.batch, "T": cfg.T, "H": cfg.H, "dtype": "f32",
               "forward_ms": timed(lambda: rnn.rnn_forward(*params, x, r)),
               "backward_sequential_ms": timed(lambda: rnn.rnn_bptt_sequential(params[0], l, d, out=s)),
               "param_grads_ms": timed(lambda: rnn.rnn_param_grads(s, d, h, x))}
        exact = rnn.rnn_bptt_sequential(params[0], l, d)
        for n in (5, 10, 20, cfg.T):
            ms = timed(lambda: rnn.rnn_bptt_jacobi(params[0], l, d, n, out=s))
            sn = rnn.rnn_bptt_jacobi(params[0], l, d, n)
            err = ((sn - exact).norm() / exact.norm()).item()
            flops = 2.0 * cfg.batch * n * cfg.T * cfg.H * cfg.H
            rec[f"backward_jacobi_{n}"] = {"ms": ms, "rel_l2_error_vs_exact": err, "tflops": flops / ms / 1e9}
        # fp32 fused multiply-add peak: SMs x 128 lanes x 2 flop x clock
        prop = torch.cuda.get_device_properties(local)
        peak = prop.multi_processor_count * 128 * 2 * 1.965e9 / 1e12
        j = rec[f"backward_jacobi_{cfg.T}"]
        rec["roofline"] = {"bound": "alu", "kernel": "rnn_bptt_jacobi_kernel", "achieved": j["tflops"], "peak": peak,
                           "unit": "TFLOP/s", "frac": j["tflops"] / peak,
                           "peak_source": "SMs x 128 fp32 lanes x 2 x 1965 MHz (nominal; derived, not measured)"}
        rec["sequences_per_s_exact_gradient"] = cfg.batch / ((rec["forward_ms"] + rec["backward_sequential_ms"] +
                                                              rec["param_grads_ms"]) / 1e3)
        if with_oracle:
            from oracle import rnn_oracle as ro
            Wn = [p_.cpu().numpy() for p_ in params]
            xs, rs = x.cpu().numpy(), r.cpu().numpy()
            k = min(cfg.batch, 8)
            t0 = time.perf_counter()
            worst = 0.0
            for i in range(k):
                f = ro.forward(*Wn, xs[i], rs[i])
                se = ro.backprop_exact(Wn[0], f["l"], f["d"])
                ro.param_grads(se, f["d"], f["h"], xs[i])
                worst = max(worst, float(np.abs(exact[i].cpu().double().numpy() - se).max() / np.abs(se).max()))
            dt = time.perf_counter() - t0
            rec["oracle"] = {"sample": f"{k} sequences, forward + exact backward + parameter gradients, numpy float64, 1 thread",
                             "sequences_per_s": k / dt, "max_rel_error_of_gpu_exact_states": worst}
        out[name] = rec
    return out


def measure_real(pkg, local: int, with_oracle: bool):
    """Continuous states with logistic conditionals (Section 5.3.1, Appendix C.3): Jacobi with the stopping
    tolerance eps on the largest change, and with eps = 0, beside the strict order on the same kernels
    (CUDA-core path, fp32).  CUDA-event means over 10 calls after 3 warm-up calls, inputs resident, L2 flushed
    between calls."""
    import torch
    out = {}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for name, cfg in si.REAL_CONFIGS.items():
        W, b = si.made_real_weights(cfg)
        lut = np.zeros(2, np.float32)
        model = pkg.Model.made(cfg.D, 2, list(cfg.H), cfg.act, cfg.prec, W, b, lut, cfg.batch)
        noise = si.draw_noise(cfg)
        d_noise = torch.from_numpy(noise).cuda()
        x = torch.empty((cfg.batch, cfg.D), dtype=torch.float32, device="cuda")
        it = torch.empty((cfg.batch,), dtype=torch.int32, device="cuda")

        def timed(fn, reps=10):
            for _ in range(3):
                fn()
            tot = 0.0
            for _ in range(reps):
                flush.fill_(1)
                a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                fn()
                e.record()
                e.synchronize()
                tot += a.elapsed_time(e)
            return tot / reps

        rec = {"batch": cfg.batch, "T": cfg.D, "hidden": list(cfg.H), "dtype": "f32", "kernel_path": "cuda-core"}
        macs = live_macs_per_sample(cfg)
        for key, eps in (("jacobi_eps", si.REAL_EPS), ("jacobi_exact", 0.0)):
            ms = timed(lambda: pkg.jacobi_sample_real(model, d_noise, None, pkg.JS_JACOBI, 0, 0, eps, x, it))
            st = model.stats()
            it_np = it.cpu().numpy()
            rec[key] = {"eps": eps, "ms_per_call": ms, "samples_per_s": cfg.batch / ms * 1e3,
                        "iters_per_sample": {"mean": float(it_np.mean()), "max": int(it_np.max()),
                                             "forward_passes": int(st.iterations)},
                        "tflops_live": 2.0 * macs * float(it_np.sum()) / ms / 1e9}
            if key == "jacobi_eps":
                x_eps, it_eps = x.cpu().numpy(), it_np
        seq = torch.empty_like(x)
        ms_seq = timed(lambda: pkg.sequential_sample_real(model, d_noise, seq), reps=3)
        rec["sequential_on_gpu"] = {"ms": ms_seq, "us_per_position": ms_seq * 1e3 / cfg.D,
                                    "largest_distance_to_jacobi_exact": float((seq - x).abs().max().item())}
        rec["speedup_vs_sequential"] = {"jacobi_eps": ms_seq / rec["jacobi_eps"]["ms_per_call"],
                                        "jacobi_exact": ms_seq / rec["jacobi_exact"]["ms_per_call"]}
        prop = torch.cuda.get_device_properties(local)
        peak = prop.multi_processor_count * 128 * 2 * 1.965e9 / 1e12
        rec["roofline"] = {"bound": "alu", "kernel": "made_generic_kernel", "achieved": rec["jacobi_eps"]["tflops_live"],
                           "peak": peak, "unit": "TFLOP/s", "frac": rec["jacobi_eps"]["tflops_live"] / peak,
                           "peak_source": "SMs x 128 fp32 lanes x 2 x 1965 MHz (nominal; derived, not measured)"}
        if with_oracle:
            from oracle import Oracle
            orc = Oracle.made(cfg.D, 2, list(cfg.H), cfg.act, cfg.prec, W, b, lut)
            k = min(cfg.batch, 32)
            t0 = time.perf_counter()
            ref = [orc.jacobi_real(noise[i], si.REAL_EPS) for i in range(k)]
            dt = time.perf_counter() - t0
            rec["oracle"] = {"sample": f"{k} of {cfg.batch} samples, jacobi with eps {si.REAL_EPS}, 1 thread, {dt:.1f} s",
                             "samples_per_s": k / dt,
                             "iters_per_sample_mean": float(np.mean([r[1] for r in ref])),
                             "gpu_iters_mean_on_same_samples": float(it_eps[:k].mean()),
                             "largest_state_difference": float(max(np.abs(ref[i][0] - x_eps[i]).max() for i in range(k)))}
        model.close()
        out[name] = rec
    return out


def oracle_sample_count(cfg, budget_s):
    cores = os.cpu_count() or 1
    per_sample_s = (14.0 if cfg.kind == "conv" else 4.0) * live_macs_per_sample(cfg) / 0.6e9
    return int(min(cfg.batch, max(1, budget_s * cores / per_sample_s)))


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

    steps = args.steps
    inputs = make_inputs(cfg)
    rec, ex = measure_workload(pkg, cfg, inputs, args.mode, args.block, steps, args.warmup, world, rank, local,
                               args.profile, args.seq, True)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    dtype = "bf16" if cfg.prec == si.PREC_BF16 else "f32"
    roof = rec["roofline"]
    if not isinstance(roof, dict):
        roof = {"bound": "alu", "achieved": None, "peak": None, "unit": "TFLOP/s", "frac": None, "traffic": None, "note": roof}
    line = {"metric": METRIC, "value": rec["samples_per_s"], "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": max(args.warmup, 3), "ms_per_step": rec["ms_per_call"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": dtype, "data": "synthetic",
            "config": config_of(cfg, args.mode, args.block, world),
            "iters_per_sample": rec["iters_per_sample"],
            "kernel_path": rec["kernel_path"],
            "tiles": rec["tiles"],
            "roofline": roof,
            "e2e": rec["e2e"],
            "gpu_launches": steps,
            "clocks": ex["clocks"]}
    for k in ("sequential_on_gpu", "speedup_vs_seq_cached", "speedup_vs_seq_skip", "speedup_vs_seq_full"):
        if k in rec:
            line[k] = rec[k]

    # ---- CPU baseline: the oracle on a bounded sample of the same workload
    if not args.no_cpu_baseline and not args.profile:
        n = min(cfg.batch, args.ref_samples)
        line["cpu_baseline"] = cpu_leg(cfg, inputs, args.mode, args.block, n, ex["samples"], ex["iters"])
        line["iters_per_sample"]["oracle_mean_on_sample"] = line["cpu_baseline"]["iters_per_sample_mean"]
        line["iters_per_sample"]["gpu_mean_on_same_samples"] = line["cpu_baseline"]["gpu_iters_mean_on_same_samples"]

    # ---- the other seeded configs, each measured the same way (fewer details), one GPU only
    if args.all_workloads and world == 1 and not args.profile:
        wl = {cfg.name: {k: v for k, v in rec.items()}}
        if "cpu_baseline" in line:
            wl[cfg.name]["oracle"] = {k: line["cpu_baseline"][k] for k in
                                      ("sample", "iters_per_sample_mean", "gpu_iters_mean_on_same_samples",
                                       "samples_differing_from_gpu")}
        del ex, inputs
        for name, other in si.CONFIGS.items():
            if name == cfg.name:
                continue
            in2 = make_inputs(other)
            r2, ex2 = measure_workload(pkg, other, in2, "jacobi", 0, max(steps, 10), args.warmup, 1, 0, local, False,
                                       "skip", False)
            if not args.no_cpu_baseline:
                n2 = oracle_sample_count(other, 4.0)
                c2 = cpu_leg(other, in2, "jacobi", 0, n2, ex2["samples"], ex2["iters"])
                r2["oracle"] = {k: c2[k] for k in ("sample", "iters_per_sample_mean", "gpu_iters_mean_on_same_samples",
                                                   "samples_differing_from_gpu")}
            wl[name] = r2
            del ex2, in2
        # the recurrent-network workload (another instance of the same triangular-system view)
        wl.update(measure_rnn(local, not args.no_cpu_baseline))
        # continuous states with a stopping tolerance
        wl.update(measure_real(pkg, local, not args.no_cpu_baseline))
        line["workloads"] = wl
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
    ap.add_argument("--one-workload", dest="all_workloads", action="store_false",
                    help="skip the `workloads` object (the other seeded configs measured beside the headline one)")
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
        args.ref_samples = max(min(cores, cfg.batch), oracle_sample_count(cfg, 15.0))
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
