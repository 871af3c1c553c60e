#!/usr/bin/env python
"""Benchmark of the WaveRNN sampling path on B200.

One "step" = one pass of the whole hot path over one batch of synthetic input: one
wrnn_sample call that generates `n_steps` 16-bit samples for every stream row of the
workload (conditioning projection, recurrent product, gates, dual softmax, draws).
Default workload: dense H = 896, bf16 weights, batch 1, 24,000 samples (1 s of audio).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload I] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is audio samples per second with inputs resident
on the device; `e2e` is the same through the host-buffer entry point (host->device copy of
the conditioning frames and device->host copy of the samples inside the timed region).
`--impl reference` times the CPU oracle (a deliberately plain program) on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1802_08435_b200 import synth  # noqa: E402

METRIC = "audio samples/sec"
UNIT = "samples/s"
SMEM_PEAK_GBS = 148 * 128 * 1.965          # 148 SMs x 128 B/clk x 1.965 GHz = 37,228 GB/s (derived, not measured)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"], bf16_tflops_sustained=d.get("bf16_tflops_sustained"),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def run_reference(args, wl):
    """The CPU oracle as it stands, on the host cores; each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import wrnn_oracle as orc
    w, masks, cond = synth.build_workload(wl)
    cores = os.cpu_count() or 1
    threads = 1 if (wl.batch == 1 or wl.dependent) else min(cores, wl.batch)      # dependent rows are generated one after the other
    # about 2-3 s of CPU work per step
    per_row_step_ms = 2.3 * (wl.H / 896.0) ** 2
    n_steps = max(16, min(wl.n_steps, int(2500.0 * threads / (per_row_step_ms * wl.batch))))
    n_steps = min(n_steps, (wl.n_frames * synth.HOP) // max(1, wl.row_stride) - 1)
    run = oracle_runner(orc, wl, w, masks, cond, threads)
    for _ in range(max(0, min(args.warmup, 1))):
        run(min(n_steps, 64))
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run(n_steps)
    dt = (time.perf_counter() - t0) / args.steps
    value = n_steps * wl.batch * samples_per_step(wl) / dt
    sample = "first %d of %d steps x %d rows of %s per step" % (n_steps, wl.n_steps, wl.batch, wl.name)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "H": wl.H, "batch": wl.batch, "n_steps": wl.n_steps, "weights": wl.dtype,
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "x_realtime_24khz": value / 24000.0,
    }
    print(json.dumps(line), flush=True)


def samples_per_step(wl):
    """Audio samples one step of one row produces: 1, or 2 for the fused subscale variant."""
    return 2 if wl.variant == 1 else 1


def oracle_runner(orc, wl, w, masks, cond, threads):
    """-> run(n_steps): the oracle of this workload's model variant on its inputs."""
    if wl.variant == 1:
        om = orc.Fs2OracleModel(w, wl.dtype)
        return lambda n: om.run(cond[0], n, seed=synth.SEED_SAMPLING, hop=synth.HOP)
    if wl.dependent and wl.net:
        from oracle import subscale_net as sn
        om = orc.OracleModel(w, wl.dtype)
        net = sn.SubscaleNet(synth.make_subscale_net(wl.batch))
        return lambda n: sn.subscale_net_run(om, net, cond, n, synth.HOP, synth.SEED_SAMPLING)
    if wl.dependent:
        om = orc.OracleModel(w, wl.dtype)
        V, b = synth.make_subscale_conv(wl.batch, wl.dependent[0])
        return lambda n: orc.subscale_dependent_run(om, cond, V, b, wl.batch, n, synth.HOP, synth.SEED_SAMPLING)
    om = orc.OracleModel(w, wl.dtype, masks, wl.block)
    return lambda n: om.run(cond, n, wl.batch, synth.SEED_SAMPLING, hop=synth.HOP, row_stride=wl.row_stride,
                            row_offset_mul=wl.row_offset_mul, threads=threads)


def cpu_baseline(wl, budget_s=12.0):
    from oracle import wrnn_oracle as orc
    w, masks, cond = synth.build_workload(wl)
    cores = os.cpu_count() or 1
    threads = 1 if (wl.batch == 1 or wl.dependent) else min(cores, wl.batch)      # dependent rows are generated one after the other
    per_row_step_ms = 2.3 * (wl.H / 896.0) ** 2
    n_steps = max(16, min(wl.n_steps, int(budget_s * 1e3 * threads / (per_row_step_ms * wl.batch))))
    n_steps = min(n_steps, (wl.n_frames * synth.HOP) // max(1, wl.row_stride) - 1)
    run = oracle_runner(orc, wl, w, masks, cond, threads)
    t0 = time.perf_counter()
    run(n_steps)
    dt = time.perf_counter() - t0
    return {"value": n_steps * wl.batch * samples_per_step(wl) / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "first %d of %d steps x %d rows of %s, once" % (n_steps, wl.n_steps, wl.batch, wl.name),
            "extrapolated": n_steps < wl.n_steps}


KERNEL_NAMES = {1: "generic", 2: "resident", 3: "batched", 4: "sparse-cluster", 5: "batched-cluster"}
FIVE_CONFIGS = [0, 1, 2, 3, 4]            # positions of the five named configurations in synth.WORKLOADS


class Ctx:
    """What every measurement of one process shares: torch, the binding, the replica group, the device and the peaks."""

    def __init__(self, torch, B, replicas, pg, rank, world, local):
        self.torch, self.B, self.replicas, self.pg = torch, B, replicas, pg
        self.rank, self.world, self.local = rank, world, local
        self.dev = torch.device("cuda", local)
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device=self.dev)      # > 126 MB L2
        self.peaks = measured_peaks()
        self._smem_gbs = None

    def smem_stream_gbs(self):
        """Measured aggregate shared-memory stream rate (16-byte loads of a resident 144 KB buffer on every SM)."""
        if self._smem_gbs is None:
            n_sms = self.torch.cuda.get_device_properties(self.dev).multi_processor_count
            self._smem_gbs = self.B.wrnn_measure_smem_stream(n_sms, 512, 144 * 1024, 2000)
        return self._smem_gbs


def n_weights(wl, fused=False):
    H, Hh = wl.H, wl.H // 2
    n_logits, n_in = (64, 12) if fused else (256, 3)
    return 3 * H * H + 2 * Hh * Hh + 2 * n_logits * Hh + 3 * n_in * H


def latency_floor(ctx, info, Hh, alg_bytes, us_per_step, note):
    """Weight bytes over the shared-memory bandwidth plus the two chip-wide exchanges a step cannot avoid (Section 2.1:
    with the model resident the remaining cost is the synchronisation between multiprocessors), the exchange measured
    live in an empty persistent kernel of the same CTA shape."""
    K = Hh if Hh % info["n_ctas"] == 0 else info["n_ctas"] * ((Hh + info["n_ctas"] - 1) // info["n_ctas"])
    try:
        t_bar_ns = ctx.B.wrnn_measure_exchange_floor(info["n_ctas"], info["n_threads"], K, 20000)
    except ctx.B.WrnnError as e:
        return {"unavailable": str(e)}
    smem_us = alg_bytes / (ctx.smem_stream_gbs() * 1e3)
    floor_us = smem_us + 2 * t_bar_ns * 1e-3
    return {"smem_us": smem_us, "t_bar_us": t_bar_ns * 1e-3, "floor_us_per_step": floor_us, "frac_of_floor": floor_us / us_per_step,
            "note": note}


def roofline(ctx, wl, info, model, n_steps, ms_per_step, cond_bytes, out_bytes):
    """The bound of the dominant (only) kernel of a call and how close the call came to it."""
    B, peaks = ctx.B, ctx.peaks
    us_per_step = ms_per_step * 1e3 / n_steps
    wbytes = info["weight_bytes_per_step"]
    fused = wl.variant == 1
    H, Hh = wl.H, wl.H // 2
    resident = info["kernel"] in (2, 4)
    # DRAM bytes of one launch, from sizes the library reports: the packed weights are read once into shared memory
    # (resident kernels) and stay there; conditioning frames in, projected gate offsets out and in again, samples out
    g_bytes = wl.batch * (wl.n_frames if wl.n_frames else 1) * 3 * H * 4
    traffic = (wbytes + cond_bytes + 2 * g_bytes + out_bytes) if resident else None
    traffic_note = ("computed: resident weight bytes loaded once per launch (%d) + conditioning (%d) + projected gate offsets "
                    "written and read (%d) + samples (%d); does not grow with the number of steps; the ncu captures in "
                    "profiles/ measured the same quantity" % (wbytes, cond_bytes, 2 * g_bytes, out_bytes)) if resident else \
                   "weights are re-read from L2 every step; DRAM traffic not modelled"
    if wl.batch >= 2:
        flops = 2.0 * wl.batch * (3 * H * H + 2 * Hh * Hh + 2 * 256 * Hh)
        ach = flops * n_steps / (ms_per_step * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "frac": ach / peaks["bf16_tflops_sustained"], "traffic": traffic, "traffic_note": traffic_note,
                "peak_source": peaks["source"] + " sustained", "algorithmic_flops_per_step": flops}
        if info["kernel"] == 2:      # the multi-stream resident kernel stamps the phases of its first CTA's first warp
            pc = B.wrnn_phase_cycles(model)
            names = B.wrnn_phase_names(model)
            roof["phase_cycles_per_step"] = {k: round(v / n_steps, 1) for k, v in zip(names, pc)}
            roof["latency_floor"] = latency_floor(
                ctx, info, Hh, n_weights(wl) * 2, us_per_step,
                "weight bytes / measured smem stream rate + 2 x measured chip-wide exchange of one stream's state half "
                "(the exchange of %d streams moves %d times the words)" % (wl.batch, wl.batch))
        return roof
    if wl.sparsity is not None:
        ach = wbytes * n_steps / (ms_per_step * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                "traffic": traffic, "traffic_note": traffic_note, "peak_source": peaks["source"], "bytes_per_step": wbytes,
                "note": "nonzero-block bytes per step over the HBM copy bandwidth (the bound the workload names); the pruned "
                        "model is resident in shared memory, see smem and latency_floor"}
        if info["kernel"] == 4:
            roof["smem"] = {"achieved": ach, "peak": ctx.smem_stream_gbs(), "unit": "GB/s", "frac": ach / ctx.smem_stream_gbs(),
                            "peak_source": "measured: 16-byte shared-memory loads on all SMs"}
            roof["latency_floor"] = latency_floor(ctx, info, Hh, wbytes, us_per_step,
                                                  "nonzero-block bytes / measured smem stream rate + 2 x measured chip-wide exchange")
        return roof
    # single stream, weights resident in shared memory: algorithmic bytes = every stored weight read once per step
    alg_bytes = n_weights(wl, fused) * (2 if wl.dtype == "bf16" else 4)
    ach = alg_bytes * n_steps / (ms_per_step * 1e-3) / 1e9
    smem = ctx.smem_stream_gbs()
    roof = {"bound": "smem", "achieved": ach, "peak": smem, "unit": "GB/s", "frac": ach / smem, "traffic": traffic,
            "traffic_note": traffic_note, "peak_source": "measured: 16-byte shared-memory loads of a resident 144 KB buffer on all SMs",
            "peak_derived": {"value": SMEM_PEAK_GBS, "how": "148 SMs x 128 B/clk x 1.965 GHz"},
            "algorithmic_bytes_per_step": alg_bytes, "resident_bytes_read_per_step": wbytes,
            "hbm_equivalent": {"achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                               "peak_source": peaks["source"]}}
    if info["kernel"] == 2:
        roof["latency_floor"] = latency_floor(ctx, info, Hh, alg_bytes, us_per_step,
                                              "weight bytes / measured smem stream rate + 2 x measured chip-wide exchange")
        pc = B.wrnn_phase_cycles(model)
        tot = float(sum(pc)) or 1.0
        names = B.wrnn_phase_names(model)
        roof["phase_cycles_per_step"] = {k: round(v / n_steps, 1) for k, v in zip(names, pc)}
        roof["wait_share"] = sum(v for k, v in zip(names, pc) if "wait" in k) / tot
    return roof


def measure(ctx, wl, *, steps, warmup, kernel, n_steps=None, e2e=True, cpu_budget_s=12.0, sample_clocks=False):
    """One workload: create the model, warm up, time `steps` calls with CUDA events (L2 flushed before each), then the
    same through the host-buffer entry point, the roofline figures and the oracle's rate.  -> dict."""
    torch, B, replicas, pg, dev = ctx.torch, ctx.B, ctx.replicas, ctx.pg, ctx.dev
    n_steps = wl.n_steps if n_steps is None else n_steps
    w, masks, cond_np = synth.build_workload(wl)
    model = B.wrnn_create(w, wl.dtype, masks, max_batch=wl.batch, kernel=kernel, block=wl.block, variant=wl.variant)
    net = None
    try:
        info = B.wrnn_launch_info(model, wl.batch)
        cond = torch.from_numpy(cond_np).to(dev)
        out = torch.zeros((wl.batch, n_steps), dtype=torch.int16, device=dev)
        # rows of different ranks are different streams of the same workload (replicas; no collective on the path)
        kw = dict(hop=synth.HOP, row_stride=wl.row_stride, row_offset_mul=wl.row_offset_mul, stream0=0)
        seed = replicas.rank_seed(synth.SEED_SAMPLING, ctx.rank)
        fused = wl.variant == 1
        if fused:       # two streams per call, then the interleaved samples (the two pre-roll samples of part B dropped)
            out = torch.zeros((2, n_steps), dtype=torch.int16, device=dev)
            u_out = torch.zeros((2 * (n_steps - 2),), dtype=torch.int16, device=dev)
        dep = wl.dependent
        if dep:
            Vn, bn = synth.make_subscale_conv(wl.batch, dep[0])
            V_d, b_d = torch.from_numpy(Vn).to(dev), torch.from_numpy(bn).to(dev)
            out = torch.zeros((wl.batch * n_steps,), dtype=torch.int16, device=dev)
            if wl.net:
                net = B.wrnn_subscale_net_create(synth.make_subscale_net(wl.batch))

        def one():
            if net is not None:
                B.wrnn_sample_subscale_net(model, net, cond, dep[0], dep[1], dep[2], wl.batch * n_steps, seed, out, hop=synth.HOP)
            elif dep:
                B.wrnn_sample_subscale_dependent(model, cond, V_d, b_d, dep[0], dep[1], dep[2], wl.batch * n_steps, wl.batch, seed, out, hop=synth.HOP)
            elif fused:
                B.wrnn_fs2_sample(model, cond, n_steps, seed, out, hop=synth.HOP)
                B.wrnn_fs2_unfold(out, n_steps, u_out)
            else:
                B.wrnn_sample(model, cond, n_steps, wl.batch, seed, out, **kw)

        for _ in range(max(warmup, 3)):
            one()
        torch.cuda.synchronize()
        assert B.wrnn_poll_status(model) == 0, B.wrnn_last_error(model)

        sampler = ClockSampler(ctx.local) if (sample_clocks and ctx.rank == 0) else None
        if sampler:
            sampler.start()
            time.sleep(0.25)
        replicas.barrier(pg)
        torch.cuda.synchronize()
        launches0 = B.wrnn_launch_count()
        evs = []
        for _ in range(steps):
            ctx.flush.fill_(1)                                            # L2 flush between timed iterations
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            one()
            e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        launches = B.wrnn_launch_count() - launches0
        replicas.barrier(pg)
        total_ms = replicas.max_over_ranks(sum(a.elapsed_time(b) for a, b in evs), pg, dev)
        clocks = sampler.stop() if sampler else None
        assert B.wrnn_poll_status(model) == 0, B.wrnn_last_error(model)

        if info["kernel"] == 2 and ctx.rank == 0:
            # the phase table comes from one extra call with the stamps switched on (they slow the stamped warp, so the
            # timed calls run without them)
            B.wrnn_phase_profile(model, True)
            one()
            torch.cuda.synchronize()
            B.wrnn_phase_profile(model, False)

        ms_per_step = total_ms / steps
        samples_per_call = 2 * (n_steps - 2) if fused else n_steps * wl.batch
        value = replicas.aggregate_throughput(ctx.world, samples_per_call, ms_per_step * 1e-3)

        # end to end through the host-buffer entry point (pinned host memory)
        e2e_d = None
        if e2e:
            cond_pin = torch.from_numpy(cond_np).pin_memory()
            out_pin = torch.zeros((2 * (n_steps - 2),) if fused else (wl.batch, n_steps), dtype=torch.int16).pin_memory()
            if dep:
                V_pin, b_pin = torch.from_numpy(Vn).pin_memory(), torch.from_numpy(bn).pin_memory()
                out_pin = torch.zeros((wl.batch * n_steps,), dtype=torch.int16).pin_memory()

            def one_host():
                if dep:      # host buffers in and out around the device entry point
                    cond.copy_(cond_pin, non_blocking=True); V_d.copy_(V_pin, non_blocking=True); b_d.copy_(b_pin, non_blocking=True)
                    one()
                    out_pin.copy_(out, non_blocking=True)
                    torch.cuda.synchronize()
                elif fused:
                    B.wrnn_fs2_sample_host(model, cond_pin.numpy()[0], n_steps, seed, out_pin.numpy(), hop=synth.HOP)
                else:
                    B.wrnn_sample_host(model, cond_pin.numpy(), n_steps, wl.batch, seed, out_pin.numpy(), **{k: v for k, v in kw.items() if k != "stream0"})

            for _ in range(2):
                one_host()
            replicas.barrier(pg)
            t0 = time.perf_counter()
            for _ in range(steps):
                one_host()
            dt = (time.perf_counter() - t0) / steps
            dt = replicas.max_over_ranks(dt, pg, dev)
            assert np.array_equal(out_pin.numpy(), (u_out if fused else out).cpu().numpy()), "host-buffer path disagrees with the device path"
            e2e_d = {"value": replicas.aggregate_throughput(ctx.world, samples_per_call, dt), "unit": UNIT,
                     "h2d_bytes_per_step": int(cond_np.nbytes) + (int(Vn.nbytes + bn.nbytes) if dep else 0),
                     "d2h_bytes_per_step": int(out_pin.numel() * 2)}

        res = {"wl": wl, "n_steps": n_steps, "info": info, "ms_per_step": ms_per_step, "value": value, "launches": int(launches),
               "clocks": clocks, "e2e": e2e_d, "samples_per_call": samples_per_call, "roofline": None, "cpu_baseline": None}
        if ctx.rank == 0:
            res["roofline"] = roofline(ctx, wl, info, model, n_steps, ms_per_step, int(cond_np.nbytes), int(out.numel() * 2))
            if cpu_budget_s and ctx.world == 1:
                res["cpu_baseline"] = cpu_baseline(wl, cpu_budget_s)
        return res
    finally:
        if net is not None:
            B.wrnn_subscale_net_destroy(net)
        B.wrnn_destroy(model)


def config_entry(res):
    """One element of the line's `configs` array."""
    wl, info = res["wl"], res["info"]
    return {"workload": wl.name, "kernel": KERNEL_NAMES[info["kernel"]], "n_ctas": info["n_ctas"], "batch": wl.batch,
            "n_steps": res["n_steps"], "us_per_step": res["ms_per_step"] * 1e3 / res["n_steps"], "value": res["value"], "unit": UNIT,
            "x_realtime_24khz": res["value"] / 24000.0, "roofline": res["roofline"], "e2e": res["e2e"],
            "cpu_baseline": res["cpu_baseline"]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=1, help="index into the workload list (default 1: dense 896 bf16, batch 1, 24000)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--n-steps", type=int, default=None, help="override samples per call (profiling of a short case)")
    ap.add_argument("--kernel", default="auto", choices=["auto", "generic", "resident", "batched", "bcluster"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the other four named configurations after the headline one")
    args = ap.parse_args()
    wl = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
        return

    from paper_1802_08435_b200 import replicas
    if replicas.needs_launch(args.gpus):
        # asked for several GPUs without a launcher: start one rank per GPU ourselves
        raise SystemExit(replicas.launch_local(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:]))
    replicas.check_world(args.gpus)

    import torch
    from paper_1802_08435_b200 import binding as B

    rank, world, local = replicas.rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    if torch.cuda.device_count() <= local:
        raise SystemExit("rank %d has no GPU of its own (%d visible)" % (rank, torch.cuda.device_count()))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    pg = replicas.init("nccl", dev)
    ctx = Ctx(torch, B, replicas, pg, rank, world, local)

    kern = {"auto": B.WRNN_KERNEL_AUTO, "generic": B.WRNN_KERNEL_GENERIC, "resident": B.WRNN_KERNEL_RESIDENT, "batched": B.WRNN_KERNEL_BATCHED, "bcluster": B.WRNN_KERNEL_BCLUSTER}[args.kernel]
    head = measure(ctx, wl, steps=args.steps, warmup=args.warmup, kernel=kern, n_steps=args.n_steps, e2e=not args.no_e2e,
                   cpu_budget_s=0.0 if args.no_cpu_baseline else 12.0, sample_clocks=True)

    # the other named configurations, each measured the same way (one GPU only: the scaling runs time the headline alone)
    configs = None
    if world == 1 and args.workload == 1 and args.n_steps is None and args.kernel == "auto" and not args.no_configs:
        sampler = ClockSampler(local)
        sampler.start()
        configs = []
        for i in FIVE_CONFIGS:
            if i == args.workload:
                configs.append(config_entry(head))
                continue
            r = measure(ctx, synth.WORKLOADS[i], steps=5, warmup=3, kernel=B.WRNN_KERNEL_AUTO, e2e=not args.no_e2e,
                        cpu_budget_s=0.0 if args.no_cpu_baseline else 4.0)
            configs.append(config_entry(r))
        configs_clocks = sampler.stop()

    if rank == 0:
        info, n_steps, ms_per_step = head["info"], head["n_steps"], head["ms_per_step"]
        line = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "H": wl.H, "batch": wl.batch, "n_steps": n_steps, "weights": wl.dtype,
                       "sparsity": wl.sparsity, "block": ("%dx%d" % tuple(wl.block)) if wl.sparsity is not None else None, "l2": "flushed between timed iterations (256 MiB fill)",
                       "kernel": KERNEL_NAMES[info["kernel"]], "n_ctas": info["n_ctas"],
                       "threads_per_cta": info["n_threads"], "smem_bytes_per_cta": info["smem_bytes"],
                       "multi_gpu": "replicas only"},
            "us_per_sample_step": ms_per_step * 1e3 / n_steps, "x_realtime_24khz": head["value"] / world / wl.batch / 24000.0 * wl.batch,
            "x_realtime_24khz_per_stream": head["samples_per_call"] / wl.batch / (ms_per_step * 1e-3) / 24000.0 * (wl.subscale_B or 1),
            "paper_context": "4x real time (96,000 samples/s) on an Nvidia P100 (Section 2.1); not the target",
            "gpu_launches": head["launches"], "clocks": head["clocks"], "roofline": head["roofline"], "e2e": head["e2e"],
        }
        if head["cpu_baseline"] is not None:
            line["cpu_baseline"] = head["cpu_baseline"]
        if configs is not None:
            line["configs"] = configs
            line["configs_clocks"] = configs_clocks
        print(json.dumps(line), flush=True)
    if pg is not None:
        pg.destroy_process_group()


if __name__ == "__main__":
    main()
