#!/usr/bin/env python
"""Benchmark of the CFGzip decode-step path on B200.

One "step" is one pass of the whole hot path over one batch: class-mask expansion, in-place
logit masking, masked log-softmax normaliser, greedy argmax and token->representative map
(one call of cfgzip_masked_logsoftmax_argmax). The default workload is the Llama-3-size
configuration: V=128256, K=2048 Zipf(1.1) classes, B=32 rows of bf16 N(0, sigma=2) logits,
class-mask density 0.1. Inputs are seeded and synthetic (module ``synth``).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl own|reference]

Prints ONE JSON line (rank 0). ``value`` is rows/s over all GPUs with inputs resident in
HBM; ``e2e`` is the same metric through the host-buffer entry point with the copies inside
the timed region; ``roofline`` relates the fused kernel to the measured HBM copy rate;
``cpu_baseline`` is the CPU oracle timed on this machine's host cores (a reported baseline,
not a target). ``--impl reference`` times only that oracle.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "masked_rows_per_s"
UNIT = "rows/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
RING_BYTES = 1 << 30          # working buffers cover at least this much, several times the 126 MB L2
RING_MAX_STEPS = 1000
RING_MAX_BYTES = 24 << 30

# DRAM traffic of the dominant (streaming) kernel per launch = per step (dram__bytes_read.sum +
# dram__bytes_write.sum from one ncu capture), keyed by workload; valid only for the kernel sources whose digest is
# recorded with it. None until a capture of the current sources exists.
NCU_TRAFFIC = {"cfg2_B32_dense": {"digest": "59571828e471fddd", "bytes_per_launch": 8539051}}


def _kernel_digest() -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2605_29986_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.endswith(".cuh"):  # the kernels; the launch shape of the headline workload is pinned by tests/test_planner.py
            h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()[:16]


def _dist_env():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def _host_threads() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(B: int, V: int, K: int, elem: int, n_partitions: int = 1, class_id_bytes: int = 2) -> int:
    """Bytes one fused dense step must move: read + write the logits, write the vocab mask, read the
    class masks, write four 4-byte results per row, read the token->class vector once per partition."""
    VW, KW = (V + 31) // 32, (K + 31) // 32
    return B * (2 * V * elem + 4 * VW + 4 * KW + 16) + n_partitions * V * class_id_bytes


# ----------------------------------------------------------------------------- clocks

class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU through NVML while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, uuid: str, period_s: float = 0.001):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples, self.reason_bits = [], 0
        self.sm_max = None
        self._halt = threading.Event()
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid if isinstance(uuid, bytes) else uuid.encode())
            self.sm_max = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._h = None

    def _read(self):
        nv = self._nv
        self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
        try:
            self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
        except Exception:
            self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))

    def run(self):
        if self._h is None:
            return
        while not self._halt.is_set():
            try:
                self._read()
            except Exception:
                break
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        self.join(timeout=2.0)
        if self._h is not None and not self.samples:
            try:
                self._read()
            except Exception:
                pass

    def summary(self) -> dict:
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "samples": 0}
        reasons = [name for bit, name in sorted(self.REASONS.items()) if self.reason_bits & bit]
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.sm_max, "reasons": reasons,
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------- workload on the device

class StepRunner:
    """A ring of resident working buffers for one workload and CUDA graphs that run steps over it."""

    def __init__(self, cz, torch, device: int, config: int, B: int = None, mode: str = "dense", steps_hint: int = 1000,
                 unique: int = 8, tune=(), unfused: bool = False, ring: int = 0, inv_temperature: float = 0.0):
        self.cz, self.torch = cz, torch
        self.unfused = unfused  # separate expand + mask calls instead of the fused step (no reductions)
        self.inv_temperature = inv_temperature  # > 0: the sampling step (cfgzip_masked_sample) instead of the greedy one
        spec = synth.CONFIGS[config]
        self.w = synth.make_workload(config, B=min(B or spec["B"], 64))  # unique rows; tiled up to B below
        self.B = B or spec["B"]
        self.V, self.K, self.dtype = self.w.V, self.w.K, self.w.dtype
        self.elem = 2 if self.dtype == "bf16" else 4
        self.VW, self.KW = (self.V + 31) // 32, (self.K + 31) // 32
        self.mode = {"dense": cz.DENSE, "sparse": cz.SPARSE, "auto": cz.AUTO}[mode]
        self.ctx = cz.cfgzip_create(device)
        for item in tune:
            name, value = item.split("=")
            cz.cfgzip_set_tuning(self.ctx, name, int(value))
        self.parts = [cz.cfgzip_load_partition(self.ctx, p.c, p.V, p.r, p.K) for p in self.w.partitions]
        ring_override = ring
        step_bytes = self.B * self.V * self.elem
        ring = max(4, -(-RING_BYTES // step_bytes))
        ring = max(ring, min(steps_hint, RING_MAX_STEPS))
        self.R = int(max(1, min(ring, RING_MAX_BYTES // step_bytes)))
        if ring_override:
            self.R = ring_override  # a short ring stays in L2: only for the figure labelled warm
        self.U = min(self.R, unique)
        # steps per CUDA graph: one pass over the ring; a short (L2-resident) ring is cycled 500 times per graph so
        # that the replay cost of a graph stays negligible there too
        self.G = self.R if not ring_override else 500 * self.R
        tile = -(-self.B // self.w.B)
        tdt = torch.int16 if self.dtype == "bf16" else torch.float32
        self.host_logits = []
        self.pristine = []
        for u in range(self.U):
            z = self.w.logits(u)
            z = np.tile(z, (tile, 1))[: self.B]
            self.host_logits.append(z)
            self.pristine.append(torch.from_numpy(z.view(np.int16) if self.dtype == "bf16" else z).cuda())
        cms = []
        for j in range(self.R):
            cm = self.w.class_masks(j)
            cms.append(np.tile(cm, (tile, 1))[: self.B])
        self.host_cm = np.stack(cms)
        self.cm = torch.from_numpy(self.host_cm.view(np.int32)).cuda()
        self.row_part_host = None if self.w.row_part is None else \
            (np.arange(self.B) % len(self.parts)).astype(np.int32)
        self.row_part = None if self.row_part_host is None else torch.from_numpy(self.row_part_host).cuda()
        self.row_part_arg = self.row_part
        if self.row_part is not None:
            # the rows keep their grammars over the steps: group them by partition once, outside the steps
            cz.cfgzip_plan_rows(self.ctx, self.parts[0], self.row_part, self.B)
            self.row_part_arg = cz.ROWS_AS_PLANNED
        self.work = torch.empty((self.R, self.B, self.V), dtype=tdt, device="cuda")
        self.vm = torch.empty((self.R, self.B, self.VW), dtype=torch.int32, device="cuda")
        self.am = torch.empty((self.R, self.B), dtype=torch.int32, device="cuda")
        self.rep = torch.empty_like(self.am)
        self.lse = torch.empty((self.R, self.B), dtype=torch.float32, device="cuda")
        self.lpa = torch.empty_like(self.lse)
        self.u = None
        if inv_temperature > 0:
            us = np.stack([np.tile(self.w.uniforms(j), tile)[: self.B] for j in range(self.R)])
            self.u = torch.from_numpy(us).cuda()
        self.stream = torch.cuda.Stream()
        self.graphs = {}
        self.launches = {}
        self.pass_events = None
        self.pass_us_per_step = []
        self.restore()

    def close(self):
        self.graphs.clear()
        self.cz.cfgzip_destroy(self.ctx)

    def restore(self):
        """Refill every working buffer with unmasked logits (outside any timed region)."""
        for j in range(self.R):
            self.work[j].copy_(self.pristine[j % self.U])
        self.torch.cuda.synchronize()

    def call(self, j: int, stream):
        cz = self.cz
        if self.unfused:
            cz.cfgzip_expand_mask(self.ctx, self.parts[0], self.row_part, self.cm[j], self.KW, self.vm[j], self.VW,
                                  self.B, self.mode, stream)
            cz.cfgzip_mask_logits(self.ctx, self.work[j], cz.BF16 if self.dtype == "bf16" else cz.F32, self.V, self.B,
                                  self.V, self.vm[j], self.VW, stream)
            return
        if self.u is not None:
            cz.cfgzip_masked_sample(
                self.ctx, self.parts[0], self.row_part_arg, self.cm[j], self.KW, self.work[j],
                cz.BF16 if self.dtype == "bf16" else cz.F32, self.V, self.B, self.vm[j], self.VW, self.u[j],
                self.inv_temperature, self.am[j], self.rep[j], self.lpa[j], self.lse[j], self.mode, stream)
            return
        cz.cfgzip_masked_logsoftmax_argmax(
            self.ctx, self.parts[0], self.row_part_arg, self.cm[j], self.KW, self.work[j],
            cz.BF16 if self.dtype == "bf16" else cz.F32, self.V, self.B, self.vm[j], self.VW, self.am[j], self.rep[j],
            self.lpa[j], self.lse[j], None, self.mode, stream)

    def graph(self, n: int):
        """CUDA graph of steps 0..n-1 of the ring (captured once per n)."""
        if n not in self.graphs:
            torch = self.torch
            g = torch.cuda.CUDAGraph()
            self.stream.wait_stream(torch.cuda.current_stream())
            before = self.cz.cfgzip_launch_count(self.ctx)
            with torch.cuda.stream(self.stream):
                with torch.cuda.graph(g, stream=self.stream):
                    for j in range(n):
                        self.call(j % self.R, self.stream)
            self.launches[n] = self.cz.cfgzip_launch_count(self.ctx) - before
            self.graphs[n] = g
        return self.graphs[n]

    def prepare(self, n_steps: int):
        full, rem = divmod(n_steps, self.G)
        if full:
            self.graph(self.G)
        if rem:
            self.graph(rem)

    def run(self, n_steps: int) -> int:
        """Enqueue n_steps steps (ring order, wrapping) on self.stream; returns kernels launched."""
        full, rem = divmod(n_steps, self.G)
        launched = 0
        with self.torch.cuda.stream(self.stream):
            for _ in range(full):
                self.graph(self.G).replay()
                launched += self.launches[self.G]
                if self.pass_events is not None:  # one event per pass over the ring, inside the timed region
                    ev = self.torch.cuda.Event(enable_timing=True)
                    ev.record(self.stream)
                    self.pass_events.append(ev)
            if rem:
                self.graph(rem).replay()
                launched += self.launches[rem]
        return launched

    def timed(self, n_steps: int, warmup: int, barrier=None, sampler: ClockSampler = None):
        """(seconds, launches) for n_steps steps after `warmup` untimed ones; events on the launching stream."""
        torch = self.torch
        self.prepare(n_steps)
        self.prepare(max(warmup, 3))
        self.run(max(warmup, 3))
        # every CUDA graph the timed region replays has run once before it (the first replay of a graph
        # also uploads it): these are extra untimed steps on top of the warm-up
        full, rem = divmod(n_steps, self.G)
        self.run((self.G if full else 0) + rem)
        self.stream.synchronize()
        self.restore()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        if barrier:
            barrier()
        if sampler:
            sampler.start()
        self.pass_events = []
        e0.record(self.stream)
        launched = self.run(n_steps)
        e1.record(self.stream)
        self.stream.synchronize()
        torch.cuda.synchronize()
        marks, self.pass_events = [e0] + self.pass_events, None
        self.pass_us_per_step = [a.elapsed_time(b) * 1e3 / self.G for a, b in zip(marks, marks[1:])]
        if sampler:
            sampler.stop()
        if barrier:
            barrier()
        return e0.elapsed_time(e1) * 1e-3, launched

    def alg_bytes(self) -> int:
        if self.mode == self.cz.SPARSE and not self.unfused:
            return self.alg_bytes_sparse()
        return algorithmic_bytes(self.B, self.V, self.K, self.elem, len(self.parts))

    def alg_bytes_sparse(self) -> int:
        """Bytes one class-list step must move: write the whole row and its vocab mask, read the class masks, and per
        allowed token read its id from the class list (4 bytes) and its logit; mean over the steps of the ring."""
        allowed_tokens = 0.0
        for j in range(min(self.R, 8)):
            bits = synth.unpack_bits(self.host_cm[j], self.K)  # [B, K]
            for b in range(self.B):
                p = self.w.partitions[0 if self.row_part_host is None else int(self.row_part_host[b])]
                allowed_tokens += float(p.sizes[bits[b]].sum())
        allowed_tokens /= min(self.R, 8)
        return int(self.B * (self.V * self.elem + 4 * self.VW + 4 * self.KW + 16) + allowed_tokens * (4 + self.elem))


def _extra_steps(runner: StepRunner, passes: int = 3, min_steps: int = 300) -> int:
    """Steps of a secondary measurement: whole passes over the ring, at least `min_steps` steps, so that the timed
    region lasts tens of milliseconds (a few milliseconds right after host-side set-up measured up to 10 % slow)."""
    return runner.R * max(passes, -(-min_steps // runner.R))


def _e2e(runner: StepRunner, torch, n_steps: int):
    """Rows/s through cfgzip_decode_step_host: pinned host inputs in, results out, every step."""
    cz = runner.cz
    pin = [torch.from_numpy(z.view(np.int16) if runner.dtype == "bf16" else z).pin_memory() for z in runner.host_logits]
    cm_pin = torch.from_numpy(runner.host_cm.view(np.int32)).pin_memory()
    B, VW = runner.B, runner.VW
    vm = torch.empty((B, VW), dtype=torch.int32).pin_memory()
    am = torch.empty(B, dtype=torch.int32).pin_memory()
    rep = torch.empty(B, dtype=torch.int32).pin_memory()
    lse = torch.empty(B, dtype=torch.float32).pin_memory()
    lpa = torch.empty(B, dtype=torch.float32).pin_memory()
    dt = cz.BF16 if runner.dtype == "bf16" else cz.F32

    def step(j):
        cz.cfgzip_decode_step_host(runner.ctx, runner.parts[0], runner.row_part_host, cm_pin[j % runner.R], runner.KW,
                                   pin[j % runner.U], dt, B, None, vm, am, rep, lpa, lse, runner.mode, runner.stream)

    for j in range(3):
        step(j)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for j in range(n_steps):
        step(j)
    torch.cuda.synchronize()
    dt_s = time.perf_counter() - t0
    h2d = B * runner.V * runner.elem + B * runner.KW * 4 + (B * 4 if runner.row_part_host is not None else 0)
    d2h = B * VW * 4 + 4 * B * 4
    return dt_s, h2d, d2h


def _cpu_baseline(runner: StepRunner, torch, budget_s: float = 12.0):
    """Time the CPU oracle on the first steps of the same workload and check the GPU results of
    those steps against it. Returns (cpu_baseline dict, parity dict)."""
    import oracle
    threads = max(1, min(_host_threads(), runner.B))
    n_max = min(runner.R, 256)
    done, spent, mismatches, max_err = 0, 0.0, 0, 0.0
    am = runner.am.cpu().numpy(); rep = runner.rep.cpu().numpy()
    lse = runner.lse.cpu().numpy(); lpa = runner.lpa.cpu().numpy()
    for j in range(n_max):
        z = runner.host_logits[j % runner.U].copy()
        t0 = time.perf_counter()
        out = oracle.decode_step(runner.w.partitions, runner.row_part_host, runner.host_cm[j], z, threads=threads)
        spent += time.perf_counter() - t0
        done += 1
        ok = np.array_equal(out["argmax"], am[j]) and np.array_equal(out["rep"], rep[j])
        vm = runner.vm[j].cpu().numpy().view(np.uint32)
        ok = ok and np.array_equal(vm, out["vocab_mask"])
        if j < 4:
            got = runner.work[j].cpu().numpy()
            ok = ok and np.array_equal(got.view(np.uint8), z.view(np.uint8))
        fin = np.isfinite(out["lse"])
        ok = ok and np.array_equal(np.isfinite(lse[j]), fin)
        if fin.any():
            err = max(np.abs(lse[j][fin] - out["lse"][fin]).max(), np.abs(lpa[j][fin] - out["logp_argmax"][fin]).max())
            max_err = max(max_err, float(err))
            ok = ok and err <= 1e-4
        mismatches += 0 if ok else 1
        if spent > budget_s:
            break
    base = {"value": done * runner.B / spent, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "first %d steps (%d rows) of the same workload, %d threads over rows" % (done, done * runner.B, threads)}
    parity = {"steps_checked": done, "mismatching_steps": mismatches, "max_abs_err_log": max_err}
    return base, parity


# ----------------------------------------------------------------------------- arms

def run_own(args):
    import torch
    from paper_2605_29986_b200 import binding as cz

    rank, local_rank, world = _dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CFGzip library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()

    runner = StepRunner(cz, torch, local_rank, args.workload, B=args.batch, mode=args.mode, steps_hint=args.steps,
                        tune=args.tune, inv_temperature=args.sample_inv_temperature)
    props = torch.cuda.get_device_properties(local_rank)
    sampler = ClockSampler("GPU-" + str(props.uuid))
    seconds, launches = runner.timed(args.steps, args.warmup, barrier, sampler)
    e2e_steps = max(3, min(args.steps, args.e2e_steps))
    barrier()
    e2e_s, h2d, d2h = _e2e(runner, torch, e2e_steps)
    if dist is not None:
        from paper_2605_29986_b200 import rows
        seconds = rows.max_over_ranks(seconds, dist, device="cuda")
        e2e_s = rows.max_over_ranks(e2e_s, dist, device="cuda")
    peak, peak_src = _measured_peak()
    alg = runner.alg_bytes()
    # a dense step is two launches (streaming kernel + per-row finalize); the figure is per step
    achieved = alg * args.steps / seconds / 1e9
    key = "cfg%d_B%d_%s" % (args.workload, runner.B, args.mode)
    traffic = None
    if key in NCU_TRAFFIC and NCU_TRAFFIC[key]["digest"] == _kernel_digest():
        traffic = NCU_TRAFFIC[key]["bytes_per_launch"]
    line = {
        "metric": METRIC, "value": world * runner.B * args.steps / seconds, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": seconds / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": runner.dtype if runner.dtype != "f32" else "f32",
        "data": "synthetic",
        "config": {
            "workload": "cfg%d %s: V=%d K=%d B=%d %s, fused expand+mask+lse+%s+rep, %s" % (
                args.workload, synth.CONFIGS[args.workload]["name"], runner.V, runner.K, runner.B, runner.dtype,
                "argmax" if not args.sample_inv_temperature else "sample(1/T=%g)" % args.sample_inv_temperature, args.mode),
            "rows_per_gpu": runner.B, "global_rows": world * runner.B,
            "l2": "inputs larger than L2: ring of %d working buffers (%.2f GB), refilled with unmasked logits before the "
                  "timed region" % (runner.R, runner.R * runner.B * runner.V * runner.elem / 1e9),
            "launch": "CUDA graph of %d steps replayed (each graph replayed once, untimed, before the timed region); "
                      "%.0f kernels per step (streaming pass + per-row finalize)" % (
                min(runner.R, args.steps), launches / max(args.steps, 1)),
            "parallelism": "rows sharded over %d GPU(s), no collective on the path" % world,
            "row_grouping": ("rows grouped by partition once before the steps (cfgzip_plan_rows), reused by every step"
                             if runner.row_part is not None else "one partition: rows grouped implicitly"),
        },
        "us_per_step": seconds / args.steps * 1e6,
        "us_per_step_over_ring_passes": (
            {"passes": len(runner.pass_us_per_step), "median": float(np.median(runner.pass_us_per_step)),
             "p10": float(np.percentile(runner.pass_us_per_step, 10)),
             "p90": float(np.percentile(runner.pass_us_per_step, 90))} if runner.pass_us_per_step else None),
        "gpu_launches": launches,
        "e2e": {"value": world * runner.B * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "what": "cfgzip_decode_step_host: pinned host logits + class masks in; vocab mask, argmax, rep, lse, "
                        "logp_argmax out; synchronised every step"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic, "peak_source": "of " + peak_src, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                     "algorithmic_bytes_per_step": alg, "launches_per_step": launches / max(args.steps, 1),
                     "kernel": ("k_step_sparse" if args.mode == "sparse" else
                                "k_step_dense_pipe (+ %s)" % ("k_sample_rows" if args.sample_inv_temperature else "k_finalize_rows"))},
        "clocks": sampler.summary(),
        "paper_context": "paper reports no timing of this path; its speedups (up to two orders of magnitude in grammar-engine "
                         "latency, up to 7.5x end to end) are for 1x H100 + Xeon Gold 6430 x16 threads, precision unstated",
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not args.sample_inv_temperature:
        line["cpu_baseline"], line["parity"] = _cpu_baseline(runner, torch)
    runner.close()
    if rank == 0 and world == 1 and not args.no_extras:
        extras = []
        for B in (128, 256, 1024):
            r2 = StepRunner(cz, torch, local_rank, args.workload, B=B, mode=args.mode, steps_hint=8, unique=2,
                            tune=args.tune)
            n = _extra_steps(r2)
            s2, l2 = r2.timed(n, r2.R)
            a2 = r2.alg_bytes() / (s2 / n) / 1e9
            extras.append({"B": B, "us_per_step": s2 / n * 1e6, "rows_per_s": B * n / s2, "achieved_gbs": a2,
                           "frac_of_measured": a2 / peak, "ring": r2.R})
            r2.close()
        line["larger_batches"] = extras
        # the same masking through the two separate calls (expand, then mask; no normaliser, argmax or map):
        # the vocab mask is written and read back, so it moves more bytes for less work
        r3 = StepRunner(cz, torch, local_rank, args.workload, B=args.batch, mode=args.mode, steps_hint=256, unique=2,
                        tune=args.tune, unfused=True)
        n = _extra_steps(r3, 2)
        s3, l3 = r3.timed(n, r3.R)
        line["unfused_expand_then_mask"] = {"us_per_step": s3 / n * 1e6, "launches_per_step": l3 / n}
        r3.close()
        # the sampling step (inverse CDF at the paper's temperature 0.2, one uniform number per row) on the same workload
        samp = []
        for B in (args.batch or synth.CONFIGS[args.workload]["B"], 1024):
            r6 = StepRunner(cz, torch, local_rank, args.workload, B=B, mode=args.mode, steps_hint=64, unique=2,
                            tune=args.tune, inv_temperature=5.0)
            n = _extra_steps(r6)
            s6, l6 = r6.timed(n, r6.R)
            samp.append({"B": B, "us_per_step": s6 / n * 1e6, "launches_per_step": l6 / n,
                         "frac_of_measured": r6.alg_bytes() / (s6 / n) / 1e9 / peak})
            r6.close()
        line["sampling_step_T0.2"] = samp
        # the same step on two buffers that stay in the 126 MB L2: NOT an HBM figure, only the latency floor
        r5 = StepRunner(cz, torch, local_rank, args.workload, B=args.batch, mode=args.mode, steps_hint=2, unique=2,
                        tune=args.tune, ring=2)
        s5, _ = r5.timed(2000, 100)
        line["warm_l2_us_per_step"] = s5 / 2000 * 1e6
        r5.close()
        # the five workloads at their own sizes (cfg2 is the headline above), same protocol, shorter runs
        five = []
        for cfg in sorted(synth.CONFIGS):
            r7 = StepRunner(cz, torch, local_rank, cfg, mode="dense", steps_hint=64, unique=2, tune=args.tune)
            n = _extra_steps(r7)
            s7, l7 = r7.timed(n, r7.R)
            a7 = r7.alg_bytes() / (s7 / n) / 1e9
            five.append({"workload": "cfg%d %s: V=%d K=%d B=%d %s, %d partition(s)" % (
                             cfg, synth.CONFIGS[cfg]["name"], r7.V, r7.K, r7.B, r7.dtype, len(r7.parts)),
                         "us_per_step": s7 / n * 1e6, "rows_per_s": r7.B * n / s7, "achieved_gbs": a7,
                         "frac_of_measured": a7 / peak, "launches_per_step": l7 / n, "ring": r7.R})
            r7.close()
        line["five_workloads_dense"] = five
        # sparse-mask stress workload (1-5 allowed classes per row): gather path against class-list scatter path
        pair = {}
        for mode in ("dense", "sparse"):
            r4 = StepRunner(cz, torch, local_rank, 5, mode=mode, steps_hint=4, unique=1, tune=args.tune)
            n = _extra_steps(r4, 4)
            s4, _ = r4.timed(n, r4.R)
            pair[mode + "_us_per_step"] = s4 / n * 1e6
            pair[mode + "_algorithmic_bytes"] = r4.alg_bytes()
            pair[mode + "_achieved_gbs_of_own_algorithmic_bytes"] = r4.alg_bytes() / (s4 / n) / 1e9
            r4.close()
        pair["workload"] = "cfg5 sparse-stress: V=128256 K=512 B=1024 f32"
        line["sparse_vs_dense"] = pair
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: each step is a bounded sample of the workload's rows."""
    rank, _, world = _dist_env()
    if rank != 0:
        return
    import oracle
    spec = synth.CONFIGS[args.workload]
    threads = max(1, min(_host_threads(), spec["B"]))
    w = synth.make_workload(args.workload, B=min(spec["B"], 64))
    z0, cm0 = w.logits(0), w.class_masks(0)
    t0 = time.perf_counter()
    oracle.decode_step(w.partitions, w.row_part, cm0, z0.copy(), threads=threads)
    t_row = (time.perf_counter() - t0) / w.B
    budget = 150.0
    rows = int(max(1, min(w.B, budget / (args.steps + args.warmup) / max(t_row, 1e-9))))
    threads = min(threads, rows)
    zs = [w.logits(u)[:rows] for u in range(2)]
    cms = [w.class_masks(j)[:rows] for j in range(8)]
    rp = None if w.row_part is None else w.row_part[:rows]

    def step(j):
        oracle.decode_step(w.partitions, rp, cms[j % 8], zs[j % 2].copy(), threads=threads)

    for j in range(args.warmup):
        step(j)
    t0 = time.perf_counter()
    for j in range(args.steps):
        step(j)
    seconds = time.perf_counter() - t0
    value = rows * args.steps / seconds
    sample = "%d of the workload's %d rows per step, %d threads over rows" % (rows, spec["B"], threads)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": seconds / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "cfg%d %s: V=%d K=%d B=%d %s, CPU oracle (expand+mask+lse+argmax+rep)" % (
            args.workload, spec["name"], w.V, w.K, spec["B"], w.dtype), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10000)
    ap.add_argument("--warmup", type=int, default=100)
    ap.add_argument("--impl", choices=["own", "reference"], default="own")
    ap.add_argument("--workload", type=int, default=2, choices=sorted(synth.CONFIGS))
    ap.add_argument("--batch", type=int, default=None, help="override the workload's row count")
    ap.add_argument("--mode", choices=["dense", "sparse", "auto"], default="dense")
    ap.add_argument("--e2e-steps", type=int, default=200)
    ap.add_argument("--tune", action="append", default=[], metavar="NAME=VALUE",
                    help="library tuning knob (see cfgzip_set_tuning); may be repeated")
    ap.add_argument("--sample-inv-temperature", type=float, default=0.0, metavar="1/T",
                    help="time the sampling step (cfgzip_masked_sample) at this inverse temperature instead of the greedy one")
    ap.add_argument("--no-extras", action="store_true", help="skip the larger-batch sweep")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.steps < 1 or args.warmup < 0:
        ap.error("--steps must be >= 1 and --warmup >= 0")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_own(args)


if __name__ == "__main__":
    main()
