#!/usr/bin/env python
"""Benchmark of the quantized-and-cached DiT sampler on B200.

One "step" = one whole trajectory of the workload: DiT-XL/2, W8A8, 50-step DDIM at 256x256, batch 16,
classifier-free guidance 1.5 (network batch 32), cache interval 2, variance compensation every step.
Metric: images per second.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload ddim50|ddim100_512]

--impl reference times the CPU oracle (oracle/, as it stands) on a bounded sample of the same workload.
With N > 1 (launched by torch.distributed.run) every rank runs its own batch on its own GPU: the samples
are independent, so there is no data-path collective; only the timing is reduced (max over ranks).
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

import synth  # noqa: E402

METRIC = "DiT-XL/2 W8A8+cache images/s (256^2, 50 steps)"
METRICS = {"ddim50": METRIC, "ddim100_512": "DiT-XL/2 W8A8+cache images/s (512^2, 100 steps)",
           "ddpm250": "DiT-XL/2 W8A8+cache images/s (256^2, 250 DDPM steps)"}
WORKLOADS = {
    # name: (config, seed key, steps, batch, guidance, interval)
    "ddim50": (synth.DIT_XL2, "ddim50_xl2", 50, 16, 1.5, 2),
    "ddim100_512": (synth.DIT_XL2_512, "ddim100_xl2_512", 100, 8, None, 3),
    # the stochastic 250-step sampler of the paper's baseline row (noise supplied as an input), W8A8 + cache
    "ddpm250": (synth.DIT_XL2, "ddim50_xl2", 250, 16, 1.5, 2),
}
STOCHASTIC = {"ddpm250"}


# DRAM bytes (read + written) per GEMM launch, from the ncu capture summarised in
# profiles/gemm_i8_layers_m8192_sections.txt: QKV 18.3 MB, proj 30.0 MB, fc1 14.9 MB, fc2 65.5 MB per launch at
# M = 8192 (the shapes of the 50-step workload); each layer is 700 of the trajectory's 2801 GEMM launches.
NCU_GEMM_DRAM_BYTES_PER_LAUNCH = 700 * (18.3e6 + 30.0e6 + 14.9e6 + 65.5e6) / 2801


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"], "bf16_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock/throttle samples during the timed region."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.file.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        busy = [s for s in sm if s > 0.5 * max(sm)] or sm
        return {"sm_mhz": float(np.median(busy)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


def workload_inputs(name):
    cfg, seed_key, steps, batch, guidance, interval = WORKLOADS[name]
    seed = synth.CONFIG_SEEDS[seed_key]
    latent = synth.normal(seed, "latent", (batch, cfg.channels, cfg.latent_side, cfg.latent_side))
    labels = synth.uniform_int(seed, "labels", (batch,), 0, cfg.num_classes)
    # VC factors: a seeded table close to 1 stands in for a fitted one (the fit is offline calibration)
    vc_table = (1.0 + 0.02 * synth.normal(seed, "vc_table", (steps, cfg.channels))).astype(np.float32)
    return cfg, seed, steps, batch, guidance, interval, latent, labels, vc_table


def rank_inputs(name, rank, world):
    """Inputs of one rank: the model (seed) is the same on every rank, the batch is the rank's own
    (rank 0 of a 1-GPU run gets exactly the workload's seeded batch)."""
    cfg, seed, steps, batch, guidance, interval, latent, labels, vc_table = workload_inputs(name)
    if world > 1:
        latent = synth.normal(seed + rank, "latent", latent.shape)
        labels = synth.uniform_int(seed + rank, "labels", labels.shape, 0, cfg.num_classes)
    return cfg, seed, steps, batch, guidance, interval, latent, labels, vc_table


def reduce_max_ms(ms, dist, device=None):
    """Slowest rank's time (the job is done when the last replica is)."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def images_per_second(world, batch, n_traj, ms):
    """Whole-job throughput: every rank finished n_traj trajectories of `batch` images in `ms`."""
    return world * batch * n_traj / (ms * 1e-3)


# ------------------------------------------------------------------------------------------ CPU oracle leg
def oracle_sample_rate(name, n_images=1, n_steps=6):
    """Times the oracle on `n_images` images for the first `n_steps` sampling steps (with n_steps = 6: three refreshes
    and three reuse steps at interval 2, two and four at interval 3: 10-15 s of CPU work) and scales the mean refresh
    and reuse times to the whole trajectory.  Returns (images/s, info)."""
    from oracle import calib, dit, sampler as osampler
    cfg, seed, steps, batch, guidance, interval, latent, labels, vc_table = workload_inputs(name)
    weights = synth.model_weights(seed, cfg)
    model = dit.make_qmodel(cfg, weights)
    lat, lab = latent[:n_images], labels[:n_images]
    t0 = np.full(n_images, float((steps - 1) * (1000 // steps)))
    scales = calib.calibrate_model(model, [(lat, t0, lab)])
    ctx = dit.Context(quant="static", scales=scales)
    stamps = []
    kind = "ddpm" if name in STOCHASTIC else "ddim"
    noise = synth.normal(seed, "noise", (n_steps, n_images) + latent.shape[1:]) if kind == "ddpm" else None
    full = osampler.SamplerConfig(steps, cache_interval=interval, guidance=guidance, vc_table=vc_table, kind=kind, noise=noise)

    class Stop(Exception):
        pass

    def on_step(i, x, reuse):
        stamps.append((time.perf_counter(), reuse))
        if i + 1 >= n_steps:
            raise Stop

    t_start = time.perf_counter()
    try:
        osampler.sample(model, ctx, full, lat, lab, on_step=on_step)
    except Stop:
        pass
    durations, prev = [], t_start
    for ts, reuse in stamps:
        durations.append((ts - prev, reuse))
        prev = ts
    t_refresh = np.mean([d for d, r in durations if not r])
    reuse_d = [d for d, r in durations if r]
    t_reuse = np.mean(reuse_d) if reuse_d else t_refresh
    n_refresh = sum(1 for i in range(steps) if i % interval == 0)
    per_traj = n_refresh * t_refresh + (steps - n_refresh) * t_reuse
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count()
    info = {"kind": "oracle", "cores": cores,
            "sample": f"{n_images} image(s) x first {n_steps} of {steps} steps (refresh {t_refresh:.2f}s, reuse {t_reuse:.2f}s), "
                      f"scaled to the full trajectory; measured {sum(d for d, _ in durations):.1f}s of CPU work",
            "seconds_measured": float(sum(d for d, _ in durations))}
    return n_images / per_traj, info


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    info = None
    t_all = time.perf_counter()
    for _ in range(max(1, min(args.steps, 2))):
        v, info = oracle_sample_rate(args.workload)
        vals.append(v)
    value = float(np.mean(vals))
    cfg, seed, steps, batch, guidance, interval, *_ = workload_inputs(args.workload)
    line = {
        "impl": "reference", "metric": METRICS.get(args.workload, METRIC), "value": value, "unit": "images/s", "n_gpus": args.gpus,
        "steps": len(vals), "warmup": 0, "ms_per_step": 1e3 * (time.perf_counter() - t_all) / len(vals),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": args.workload, "model": "DiT-XL/2", "batch": batch, "sampling_steps": steps,
                   "cache_interval": interval, "guidance": guidance, "vc": "k_table every step"},
        "cpu_baseline": {"value": value, "unit": "images/s", **{k: info[k] for k in ("cores", "kind", "sample")}},
        "e2e": {"value": value, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------ CUDA leg
def run_ours(args):
    import torch
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
    import paper_2503_02508_b200 as q

    cfg, seed, steps, batch, guidance, interval, latent, labels, vc_table = rank_inputs(args.workload, rank, world)
    stream = torch.cuda.Stream()
    ctx = q.qdit_create(local, stream.cuda_stream)
    weights = synth.model_weights(seed, cfg)
    model = q.qdit_model_create(ctx, cfg, weights, args.weight_bits)
    del weights
    sampler = q.qdit_sampler_create(ctx, model, batch=batch, num_steps=steps, cache_interval=interval,
                                    use_cfg=guidance is not None, guidance=guidance or 1.0,
                                    vc_mode=q.QDIT_VC_K_TABLE, vc_table=vc_table)
    # activation ranges: on-device calibration on the starting latents at three noise levels
    beff = batch * (2 if guidance is not None else 1)
    lat_d = torch.from_numpy(latent).cuda()
    lab_d = torch.from_numpy(labels.astype(np.int32)).cuda()
    lat_eff = torch.cat([lat_d, lat_d]) if guidance is not None else lat_d
    y_eff = torch.cat([lab_d, torch.full_like(lab_d, cfg.num_classes)]) if guidance is not None else lab_d
    net = torch.empty((beff, 2 * cfg.channels, cfg.latent_side, cfg.latent_side), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    q.qdit_model_begin_calibration(ctx, model)
    for tval in (980.0, 500.0, 20.0):
        t_d = torch.full((beff,), tval, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()     # t_d is filled on torch's stream, the library reads it on its own
        q.qdit_forward(ctx, sampler, lat_eff, t_d, y_eff, beff, net, q.QDIT_FWD_CALIBRATE)
        q.qdit_sync(ctx)
    q.qdit_model_finish_calibration(ctx, model)
    q.qdit_sync(ctx)

    if args.workload in STOCHASTIC:
        gen = torch.Generator(device="cuda")
        gen.manual_seed(seed + rank)
        noise_d = torch.randn((steps, batch, cfg.channels, cfg.latent_side, cfg.latent_side), generator=gen,
                              dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()     # the noise is drawn on torch's stream, the library reads it on its own
        q.qdit_sampler_set_ddpm(ctx, sampler, noise_d)

    def trajectory_device():
        q.qdit_sampler_reset(ctx, sampler, lat_d, lab_d)
        for i in range(steps):
            q.qdit_sample_step(ctx, sampler, i)

    lat_h = torch.from_numpy(latent).pin_memory()
    lab_h = torch.from_numpy(labels.astype(np.int32)).pin_memory()
    out_h = torch.empty_like(lat_h).pin_memory()

    def trajectory_host():
        q.qdit_sample(ctx, sampler, lat_h, lab_h, out_h)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, n):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        q.qdit_sync(ctx)
        barrier()
        return reduce_max_ms(e0.elapsed_time(e1), dist, "cuda")

    n_warm = args.warmup if args.short_warmup else max(args.warmup, 3)
    for _ in range(n_warm):
        trajectory_device()
    q.qdit_sync(ctx)
    clocks = ClockSampler(local)
    clocks.start()
    l0 = q.qdit_launch_count(ctx)
    ms = timed(trajectory_device, args.steps)
    launches = q.qdit_launch_count(ctx) - l0
    clock_info = clocks.stop()
    value = images_per_second(world, batch, args.steps, ms)

    trajectory_host()
    ms_e2e = timed(trajectory_host, args.steps)
    e2e_value = images_per_second(world, batch, args.steps, ms_e2e)
    final = out_h.numpy()
    if not np.isfinite(final).all():
        raise SystemExit("non-finite latent after sampling")

    # roofline of the dominant kernel (the int8 GEMM): one extra trajectory with per-launch CUDA events
    peaks = measured_peaks()
    q.qdit_profile_enable(ctx, 1)
    trajectory_device()
    prof = {k: q.qdit_profile_read(ctx, k) for k in range(q.QDIT_PROF_KINDS)}
    q.qdit_profile_enable(ctx, 0)
    g_n, g_ms, g_ops = prof[q.QDIT_PROF_GEMM]
    int8_peak = 2.0 * peaks["bf16_sustained"]          # dense int8 : bf16 nominal ratio 4.5 : 2.25
    achieved = g_ops / (g_ms * 1e-3) / 1e12 if g_ms > 0 else 0.0
    roofline = {"bound": "tensor", "kernel": "int8 GEMMs (gemm_i8_t_kernel, gemm_i8_kernel)", "achieved": achieved,
                "peak": int8_peak, "unit": "TOP/s", "frac": achieved / int8_peak, "frac_of_nominal_4500": achieved / 4500.0,
                "traffic": NCU_GEMM_DRAM_BYTES_PER_LAUNCH if args.workload == "ddim50" else None,
                "traffic_note": "launch-weighted mean of the four block-level layers at M = 8192 (ncu, L2-warm sweep)",
                "peak_source": f"2 x {peaks['source']} sustained bf16 ({peaks['bf16_sustained']} TFLOP/s)",
                "launches": g_n, "avg_launch_ms": g_ms / max(g_n, 1), "share_of_profiled_time": None}
    tot_ms = sum(v[1] for v in prof.values())
    if tot_ms > 0:
        roofline["share_of_profiled_time"] = g_ms / tot_ms
    kinds = ["gemm", "attention", "ln_modulate", "act_quant", "cache_reuse", "other"]
    breakdown = {}
    for k, name in enumerate(kinds):
        n, t, w = prof[k]
        if n:
            rate = w / (t * 1e-3)
            breakdown[name] = {"launches": n, "ms": round(t, 3),
                               "rate": round(rate / 1e12, 2) if k < 2 else round(rate / 1e9, 1),
                               "unit": "TOP/s" if k == 0 else "TFLOP/s" if k == 1 else "GB/s",
                               "avg_us": round(1e3 * t / n, 2)}

    # the metric's second half: the GEMM layers and the memory-bound kernels alone, at the workload's row count and at
    # one larger than L2 (rank 0 of a single-GPU run only; a few seconds)
    sweep = None
    if rank == 0 and world == 1 and not args.no_sweep:
        sclk = ClockSampler(local)
        sclk.start()
        srows = sweep_rows(q, ctx, [8192, 65536], 10, peaks, stream)
        sweep = compact_sweep(srows, sclk.stop(), peaks)
        for name, b in breakdown.items():
            if name == "cache_reuse":
                sweep["memory_bound"].append({"kernel": "cache_reuse_all (inside the trajectory, 1.06 GB per launch)",
                                              "gbs": b["rate"], "frac_of_hbm": round(b["rate"] / peaks["hbm_gbs"], 3)})

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, info = oracle_sample_rate(args.workload)
        cpu = {"value": v, "unit": "images/s", "cores": info["cores"], "kind": info["kind"], "sample": info["sample"]}

    if rank == 0:
        line = {
            "metric": METRICS.get(args.workload, METRIC).replace("W8A8", f"W{args.weight_bits}A8"), "value": value, "unit": "images/s", "n_gpus": world, "steps": args.steps,
            "warmup": n_warm, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": args.workload, "model": "DiT-XL/2", "batch_per_gpu": batch, "network_batch": beff,
                       "sampling_steps": steps, "cache_interval": interval, "guidance": guidance,
                       "vc": "k_table every step", "residual_stream": "bf16", "weight_bits": args.weight_bits,
                       "sampler": "ddpm (noise supplied)" if args.workload in STOCHASTIC else "ddim",
                       "l2": "per-step working set (0.45 GB weights + 1.06 GB cache) exceeds L2; no flush needed",
                       "roofline_pass": "one extra trajectory with per-launch CUDA events, outside the timed region"},
            "clocks": clock_info,
            "e2e": {"value": e2e_value, "unit": "images/s", "h2d_bytes_per_step": int(lat_h.numel() * 4 + lab_h.numel() * 4),
                    "d2h_bytes_per_step": int(out_h.numel() * 4), "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": int(launches),
            "roofline": roofline,
            "kernels": breakdown,
            "sweep": sweep,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    q.qdit_sampler_destroy(sampler)
    q.qdit_model_destroy(model)
    q.qdit_destroy(ctx)
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------ GEMM sweep
GEMM_SHAPES = [(1152, 3456, "qkv"), (1152, 1152, "proj"), (1152, 4608, "fc1"), (4608, 1152, "fc2")]


def sweep_rows(q, ctx, ms_list, steps, peaks, stream=None):
    """Times the block's four linear layers (with the epilogue each has in the model), the activation quantizer,
    LayerNorm-modulate-quantize and attention at the given row counts.  Activations: bf16 N(0,1) with 1 % of the
    channels scaled x20; weights: int8 with channel-wise scales.  Launches are repeated back to back on the same
    operands (L2-warm below about 100 MB of operands, streaming from HBM above).  `stream`: the torch stream the
    context launches on (None: the default stream); the timing events are recorded there."""
    import torch
    seed = synth.CONFIG_SEEDS["gemm_sweep"]
    rows = []
    for M in ms_list:
        for K, N, name in GEMM_SHAPES:
            x = torch.from_numpy(synth.outlier_activations(seed, f"x{M}.{K}", M, K)).cuda().to(torch.bfloat16)
            wq = torch.from_numpy(synth.uniform_int(seed, f"w{N}.{K}", (N, K), -127, 128).astype(np.int8)).cuda()
            ws = torch.from_numpy(np.abs(synth.normal(seed, f"ws{N}", (N,), 1e-3)) + 1e-4).cuda()
            bias = torch.from_numpy(synth.normal(seed, f"b{N}", (N,), 0.02)).cuda()
            gate = torch.from_numpy(synth.normal(seed, f"g{N}", ((M + 255) // 256, N), 0.3)).cuda()
            resid = torch.from_numpy(synth.normal(seed, f"r{M}.{N}", (M, N))).cuda().to(torch.bfloat16)
            cache = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            a8 = torch.empty((M, K), dtype=torch.uint8, device="cuda")
            a_qp = q.qparams(float(x.abs().max()) / 127.0)
            if name == "qkv":
                flags, out = q.QDIT_EPI_BIAS | q.QDIT_EPI_OUT_BF16, torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            elif name == "fc1":
                flags, out = q.QDIT_EPI_BIAS | q.QDIT_EPI_GELU | q.QDIT_EPI_QUANT_OUT, torch.empty((M, N), dtype=torch.uint8, device="cuda")
            else:
                flags = q.QDIT_EPI_BIAS | q.QDIT_EPI_GATE | q.QDIT_EPI_RESIDUAL | q.QDIT_EPI_CACHE_STORE | q.QDIT_EPI_OUT_BF16
                out = resid
            epi = q.epilogue(w_scale=ws, bias=bias, gate=gate, ld_gate=N, tokens_per_sample=256, residual=resid,
                             cache_out=cache, out_qp=q.qparams(0.05))

            def quant():
                q.qdit_quantize_act(ctx, x, q.QDIT_BF16, M, K, K, q.QDIT_QUANT_STATIC, a_qp, None, a8, K)

            def gemm():
                q.qdit_w8a8_linear(ctx, a8, wq, M, N, K, a_qp, None, flags, epi, out, N)

            def both():
                quant()
                gemm()

            def t(fn):
                for _ in range(3):
                    fn()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(steps):
                    fn()
                e1.record(stream)
                torch.cuda.synchronize()
                return e0.elapsed_time(e1) / steps

            torch.cuda.synchronize()   # the operands were made on torch's stream
            quant()
            ops = 2.0 * M * N * K
            ms_g, ms_b, ms_q = t(gemm), t(both), t(quant)
            row = {"layer": name, "M": M, "K": K, "N": N, "gemm_tops": ops / ms_g / 1e9, "quant_gemm_tops": ops / ms_b / 1e9,
                   "gemm_us": ms_g * 1e3, "act_quant_gbs": 3.0 * M * K / ms_q / 1e6,
                   "act_quant_frac_of_hbm": 3.0 * M * K / ms_q / 1e6 / peaks["hbm_gbs"],
                   "frac_of_2x_bf16_burst": ops / ms_g / 1e9 / (2 * peaks["bf16_burst"]),
                   "frac_of_nominal_4500": ops / ms_g / 1e9 / 4500.0}
            if name == "qkv" and M % 256 == 0:
                # the block's other memory-bound kernel on the same tokens: LayerNorm + adaLN modulate + quantize
                mod = torch.from_numpy(synth.normal(seed, f"mod{M}", (M // 256, 6 * K), 0.3)).cuda()

                def ln():
                    q.qdit_adaln_modulate(ctx, x, M, K, 256, 1e-6, mod, mod[:, K:], 6 * K, a8, q.QDIT_I8, a_qp)

                ms_l = t(ln)
                row["ln_modulate_us"] = ms_l * 1e3
                row["ln_modulate_gbs"] = 3.0 * M * K / ms_l / 1e6
                row["ln_modulate_frac_of_hbm"] = row["ln_modulate_gbs"] / peaks["hbm_gbs"]
                # and the block's attention on the layer's output shape (16 heads of 72, 256 tokens per image)
                qkv_t = torch.from_numpy(synth.normal(seed, f"qkv{M}", (M, N))).cuda().to(torch.bfloat16)

                def attn():
                    p0 = qkv_t.data_ptr()
                    q.qdit_attention(ctx, p0, p0 + 2 * K, p0 + 4 * K, N, M // 256, 16, 256, K // 16, 1.0 / np.sqrt(K // 16),
                                     a8, q.QDIT_I8, a_qp)

                ms_a = t(attn)
                row["attention_us"] = ms_a * 1e3
                row["attention_tflops"] = 4.0 * (M // 256) * 16 * 256 * 256 * (K // 16) / ms_a / 1e9
            rows.append(row)
            del x, wq, resid, cache, a8, out
    return rows


def run_gemm_sweep(args):
    """int8 GEMM + fused activation-quantizer sweep over the DiT-XL/2 linear shapes (K -> N) and M.
    Reports TOP/s of the GEMM alone (epilogue of that layer in the model) and of act-quant + GEMM."""
    import paper_2503_02508_b200 as q
    peaks = measured_peaks()
    ctx = q.qdit_create(0, None)
    clocks = ClockSampler(0)
    clocks.start()
    rows = sweep_rows(q, ctx, args.m, args.steps, peaks)
    clock_info = clocks.stop()
    q.qdit_sync(ctx)
    q.qdit_destroy(ctx)
    best = max(r["gemm_tops"] for r in rows)
    print(json.dumps({"metric": "int8 GEMM TOP/s (DiT-XL/2 linear shapes)", "value": best, "unit": "TOP/s", "n_gpus": 1,
                      "steps": args.steps, "warmup": 3, "higher_is_better": True, "dtype": "int8", "data": "synthetic",
                      "config": {"workload": "gemm_sweep", "l2": "repeated launches on the same operands (L2-warm)"},
                      "clocks": clock_info,
                      "peaks": {"int8_2x_bf16_burst": 2 * peaks["bf16_burst"], "int8_nominal": 4500.0,
                                "hbm_gbs": peaks["hbm_gbs"], "source": peaks["source"]},
                      "rows": rows}))


def run_w4_sweep(args):
    """Packed 4-bit weights against one code per byte on the weight-streaming shapes: the stacked modulation GEMM of a
    50-step trajectory (M = 1600, N = 28 x 6912, K = 1152) and the four block layers at M = 256 and 1024.  The W4A8
    rows widen the weights inside the GEMM kernel (no scratch matrix)."""
    import torch
    import paper_2503_02508_b200 as q
    seed = synth.CONFIG_SEEDS["gemm_sweep"]
    peaks = measured_peaks()
    ctx = q.qdit_create(0, None)
    shapes = [(1600, 28 * 6912, 1152, "modulation (all blocks, 50 steps)")]
    for M in (256, 1024):
        shapes += [(M, N, K, name) for K, N, name in GEMM_SHAPES]
    rows = []
    for M, N, K, name in shapes:
        codes = synth.uniform_int(seed, f"w4.{N}.{K}", (N, K), -7, 8).astype(np.int8)
        w8 = torch.from_numpy(codes).cuda()
        w4 = torch.empty((N, K // 2), dtype=torch.uint8, device="cuda")
        q.qdit_pack_weight_int4(ctx, w8, N, K, w4)
        a8 = torch.from_numpy(synth.uniform_int(seed, f"a.{M}.{K}", (M, K), -127, 128).astype(np.int8)).cuda()
        ws = torch.from_numpy(np.abs(synth.normal(seed, f"ws{N}", (N,), 1e-3)) + 1e-4).cuda()
        bias = torch.from_numpy(synth.normal(seed, f"b{N}", (N,), 0.02)).cuda()
        out = torch.empty((M, N), dtype=torch.float32, device="cuda")
        epi = q.epilogue(w_scale=ws, bias=bias)
        flags = q.QDIT_EPI_BIAS | q.QDIT_EPI_OUT_F32
        qp = q.qparams(0.03)

        def t(fn):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / args.steps

        ms8 = t(lambda: q.qdit_w8a8_linear(ctx, a8, w8, M, N, K, qp, None, flags, epi, out, N))
        ms4 = t(lambda: q.qdit_w4a8_linear(ctx, a8, w4, M, N, K, qp, None, flags, epi, out, N, None))
        rows.append({"layer": name, "M": M, "N": N, "K": K, "w8a8_us": round(ms8 * 1e3, 1), "w4a8_us": round(ms4 * 1e3, 1),
                     "speedup": round(ms8 / ms4, 3), "weight_mb_w8": round(N * K / 1e6, 1), "weight_mb_w4": round(N * K / 2e6, 1),
                     "w4_weight_gbs": round(N * K / 2 / ms4 / 1e6, 0)})
    q.qdit_destroy(ctx)
    print(json.dumps({"metric": "W4A8 (packed) vs W8A8 linear layer time on weight-streaming shapes", "value": rows[0]["speedup"],
                      "unit": "x (modulation GEMM)", "n_gpus": 1, "steps": args.steps, "warmup": 3, "higher_is_better": True,
                      "dtype": "int8", "data": "synthetic", "config": {"workload": "w4_sweep", "output": "f32 + bias"},
                      "hbm_gbs": peaks["hbm_gbs"], "rows": rows}))


def run_mma_probe(args):
    """What the tensor pipe gives the int8 GEMM kernels at most: tcgen05.mma kind::i8 (M 128, K 32) issued by one thread
    per SM, with the operands resident in shared memory (the instruction path alone) and with a TMA producer refilling
    a four-stage ring from an L2-resident matrix as the GEMM kernels' main loop does, no epilogue."""
    import torch
    import paper_2503_02508_b200 as q
    peaks = measured_peaks()
    ctx = q.qdit_create(0, None)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rows_op = 4096
    operands = torch.randint(-127, 128, (rows_op, 1024), dtype=torch.int8, device="cuda")
    torch.cuda.synchronize()
    iters = 8192
    clocks = ClockSampler(0)
    clocks.start()
    rows = []
    for mode, name in ((0, "operands resident in shared memory"), (1, "TMA-fed four-stage ring, no epilogue")):
        for n in (128, 192, 256):
            for _ in range(3):
                q.qdit_probe_mma_rate(ctx, mode, n, iters, operands, rows_op)
            ms = min(q.qdit_probe_mma_rate(ctx, mode, n, iters, operands, rows_op) for _ in range(max(args.steps, 3)))
            ops = sms * iters * 4 * 2.0 * 128 * n * 32
            us_per_group = ms * 1e3 / iters
            rows.append({"mode": name, "n": n, "ms": round(ms, 3), "tops": round(ops / ms / 1e9, 0),
                         "us_per_128_byte_k_block": round(us_per_group, 3),
                         "frac_of_2x_bf16_burst": round(ops / ms / 1e9 / (2 * peaks["bf16_burst"]), 3),
                         "frac_of_nominal_4500": round(ops / ms / 1e9 / 4500.0, 3)})
    clock_info = clocks.stop()
    q.qdit_destroy(ctx)
    best = max(r["tops"] for r in rows if r["n"] == 256)
    print(json.dumps({"metric": "tcgen05.mma kind::i8 rate, all SMs (probe)", "value": best, "unit": "TOP/s", "n_gpus": 1,
                      "steps": max(args.steps, 3), "warmup": 3, "higher_is_better": True, "dtype": "int8", "data": "synthetic",
                      "config": {"workload": "mma_probe", "iters": iters, "timing": "CUDA events around one launch, best of steps"},
                      "clocks": clock_info, "int8_peak_2x_bf16_burst": 2 * peaks["bf16_burst"], "rows": rows}))


def compact_sweep(rows, clock_info, peaks):
    """The second half of the metric for the default bench line: per layer and M the GEMM rate and its fractions of
    2 x burst bf16 (measured) and of the nominal 4500 TOP/s; the memory-bound kernels as fractions of the measured HBM
    copy bandwidth."""
    out = {"clocks": clock_info, "int8_peak_2x_bf16_burst": 2 * peaks["bf16_burst"], "int8_nominal": 4500.0,
           "hbm_gbs": peaks["hbm_gbs"], "gemm": [], "memory_bound": [],
           "note": "launches repeated back to back on the same operands: L2-warm at M = 8192, streaming from HBM at M = 65536"}
    for r in rows:
        out["gemm"].append({"layer": r["layer"], "M": r["M"], "us": round(r["gemm_us"], 1), "tops": round(r["gemm_tops"], 0),
                            "frac_2x_bf16_burst": round(r["frac_of_2x_bf16_burst"], 3),
                            "frac_nominal": round(r["frac_of_nominal_4500"], 3),
                            "with_act_quant_tops": round(r["quant_gemm_tops"], 0)})
        if r["layer"] in ("qkv", "fc2"):
            out["memory_bound"].append({"kernel": "act_quant", "M": r["M"], "K": r["K"], "gbs": round(r["act_quant_gbs"], 0),
                                        "frac_of_hbm": round(r["act_quant_frac_of_hbm"], 3)})
        if "ln_modulate_gbs" in r:
            out["memory_bound"].append({"kernel": "ln_modulate_q8", "M": r["M"], "K": r["K"], "us": round(r["ln_modulate_us"], 1),
                                        "gbs": round(r["ln_modulate_gbs"], 0), "frac_of_hbm": round(r["ln_modulate_frac_of_hbm"], 3)})
            out.setdefault("attention", []).append({"M": r["M"], "us": round(r["attention_us"], 1),
                                                    "tflops": round(r["attention_tflops"], 0)})
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="ddim50", choices=sorted(WORKLOADS) + ["gemm_sweep", "w4_sweep", "mma_probe"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the per-layer sweep that follows the timed region")
    ap.add_argument("--weight-bits", type=int, default=8, help="code width of the quantized weights (4 = the paper's W4A8 setting)")
    ap.add_argument("--m", type=lambda v: [int(x) for x in v.split(",")], default=[256, 1024, 4096, 8192, 16384, 65536],
                    help="row counts of the GEMM sweep")
    ap.add_argument("--short-warmup", action="store_true",
                    help="profiling runs only: honour --warmup below 3 (such a run is not a valid measurement)")
    args = ap.parse_args()
    if args.workload == "gemm_sweep":
        run_gemm_sweep(args)
    elif args.workload == "w4_sweep":
        run_w4_sweep(args)
    elif args.workload == "mma_probe":
        run_mma_probe(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
