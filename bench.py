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
not a target); ``parity`` compares GPU results with that oracle. ``--impl reference`` times
only the oracle. With ``--gpus N`` > 1 and no launcher in the environment the script starts
N ranks of itself (one per GPU).

The timed region always consists of whole passes over the ring of working buffers and lasts
at least 20 ms: ``steps`` echoes the request, ``timed_steps`` is what was timed.
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
from paper_2605_29986_b200 import rows as ranks  # noqa: E402  (host-only helpers: no CUDA needed to import)

METRIC = "masked_rows_per_s"
UNIT = "rows/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
RING_BYTES = 1 << 30          # working buffers cover at least this much, several times the 126 MB L2
RING_MAX_STEPS = 1000
RING_MAX_BYTES = 24 << 30
MIN_TIMED_SECONDS = 0.02      # shorter regions read slow: the replay cost of a graph sits inside them
LOG_TOL = 1e-4                # absolute, fp32-accumulated log quantities against the fp64 oracle

# DRAM traffic of the dominant (streaming) kernel per launch = per step (dram__bytes_read.sum +
# dram__bytes_write.sum from one ncu capture, see profiles/), keyed by workload; valid only for the kernel
# sources whose digest is recorded with it. A workload without a capture of the current sources reports null.
_CAPTURED = "02183c84a4d7b29e"
NCU_TRAFFIC = {
    "cfg2_B32_dense": {"digest": _CAPTURED, "bytes_per_launch": 14954837},      # 8.24 MB read + 6.71 MB written (L2 still filling)
    "cfg2_B1024_dense": {"digest": _CAPTURED, "bytes_per_launch": 541736960},   # 263.2 MB read + 278.5 MB written
    "cfg4_B256_dense": {"digest": _CAPTURED, "bytes_per_launch": 269750784},    # 132.4 MB read + 137.4 MB written
    "cfg5_B1024_dense": {"digest": _CAPTURED, "bytes_per_launch": 1067131051},  # 526.5 MB read + 540.6 MB written
    "cfg5_B1024_sparse": {"digest": _CAPTURED, "bytes_per_launch": 611983872},  # 65.1 MB read + 546.9 MB written
}


def _kernel_digest() -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2605_29986_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.endswith(".cuh"):  # the kernels; the launch shape of the headline workload is pinned by tests/test_planner.py
            h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()[:16]


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


# ----------------------------------------------------------------------------- step and slot bookkeeping

def ring_steps(step_bytes: int, steps_hint: int) -> int:
    """Working buffers in the ring: at least RING_BYTES of logits (several times L2), at least min(steps_hint,
    RING_MAX_STEPS) buffers, never more than RING_MAX_BYTES."""
    ring = max(4, -(-RING_BYTES // step_bytes))
    ring = max(ring, min(steps_hint, RING_MAX_STEPS))
    return int(max(1, min(ring, RING_MAX_BYTES // step_bytes)))


def timed_steps_for(requested: int, steps_per_pass: int, pass_seconds: float, min_seconds: float = MIN_TIMED_SECONDS) -> int:
    """Steps the timed region runs: whole passes over the ring, at least the requested steps, at least min_seconds."""
    passes = max(1, -(-requested // steps_per_pass))
    if pass_seconds > 0:
        passes = max(passes, int(np.ceil(min_seconds / pass_seconds)))
    return passes * steps_per_pass


def spread(n: int, k: int) -> list:
    """k indices spread evenly over range(n) (all of them when k >= n), ascending and distinct."""
    if k >= n:
        return list(range(n))
    return sorted(set(int(x) for x in np.linspace(0, n - 1, k)))


def check_slots(runner, slots, row_ids=None, threads: int = 1, budget_s: float = 30.0, full_logits: int = 2) -> dict:
    """Parity of ring slots against the CPU oracle. `runner.execute_slots(slots, rows)` runs exactly these steps
    once more (untimed, on freshly refilled buffers) and returns the outputs of the chosen rows, so no slot is
    compared that was not executed. Rows `row_ids` (all when None) of each slot are compared: vocab mask, argmax
    and representative bit for bit, lse and logp_argmax within LOG_TOL, and the masked logits bit for bit on the
    first `full_logits` slots. Stops early when the oracle has used `budget_s` seconds."""
    import oracle
    slots = list(slots)
    rows_sel = np.arange(runner.B) if row_ids is None else np.asarray(sorted(row_ids), dtype=np.int64)
    got = runner.execute_slots(slots, rows_sel, full_logits)
    rp = None if runner.row_part_host is None else runner.row_part_host[rows_sel]
    checked, mismatches, max_err, spent = 0, 0, 0.0, 0.0
    for n, j in enumerate(slots):
        z = np.ascontiguousarray(runner.host_logits_of(j)[rows_sel]).copy()
        t0 = time.perf_counter()
        want = oracle.decode_step(runner.partitions, rp, np.ascontiguousarray(runner.host_cm[j][rows_sel]), z,
                                  threads=threads)
        spent += time.perf_counter() - t0
        ok = np.array_equal(got["argmax"][n], want["argmax"]) and np.array_equal(got["rep"][n], want["rep"])
        ok = ok and np.array_equal(got["vocab_mask"][n], want["vocab_mask"])
        if n < full_logits:
            ok = ok and np.array_equal(got["logits"][n].view(np.uint8), z.view(np.uint8))
        for key in ("lse", "logp_argmax"):
            g = got[key][n].astype(np.float64)
            fin = np.isfinite(want[key])
            ok = ok and np.array_equal(np.isfinite(g), fin)
            if fin.any():
                err = float(np.abs(g[fin] - want[key][fin]).max())
                max_err = max(max_err, err)
                ok = ok and err <= LOG_TOL
        checked += 1
        mismatches += 0 if ok else 1
        if spent > budget_s:
            break
    return {"steps_checked": checked, "of_ring_steps": runner.R, "rows_per_step": int(len(rows_sel)), "of_rows": runner.B,
            "mismatching_steps": mismatches, "max_abs_err_log": max_err, "tolerance_log": LOG_TOL,
            "what": "steps re-run untimed on refilled buffers, compared with the CPU oracle: vocab mask, argmax, rep bit-exact "
                    "(masked logits too on the first %d), lse and logp_argmax within the tolerance" % full_logits}


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
    """A ring of resident working buffers for one workload and a CUDA graph that runs one pass of steps over it."""

    def __init__(self, cz, torch, device: int, config: int, B: int = None, mode: str = "dense", steps_hint: int = 1000,
                 unique: int = 8, tune=(), kind: str = "fused", ring: int = 0, inv_temperature: float = 0.0, top_k: int = 0,
                 top_p: float = 1.0, allow_all: bool = False):
        self.cz, self.torch = cz, torch
        # kind: "fused" the whole step; "unfused" separate expand + mask calls (no reductions); "floor" the in-place
        # read-modify-write kernel over the same buffers (what a pass over these bytes costs at least)
        self.kind = kind
        self.inv_temperature = inv_temperature  # > 0: the sampling step (cfgzip_masked_sample) instead of the greedy one
        self.top_k, self.top_p = top_k, top_p   # sampling step: restricted to the most probable tokens when set
        spec = synth.CONFIGS[config]
        self.B = B or spec["B"]
        wl = synth.make_workload(config, B=min(self.B, 64))  # unique logits rows; tiled up to B below
        # every row has its own class mask (and partition) at every batch size; only the logits rows repeat
        self.w = wl if self.B <= 64 else synth.make_workload(config, B=self.B)
        self.partitions = self.w.partitions
        self.V, self.K, self.dtype = self.w.V, self.w.K, self.w.dtype
        self.elem = 2 if self.dtype == "bf16" else 4
        self.VW, self.KW = (self.V + 31) // 32, (self.K + 31) // 32
        self.mode_name = mode
        self.mode = {"dense": cz.DENSE, "sparse": cz.SPARSE, "auto": cz.AUTO}[mode]
        self.ctx = cz.cfgzip_create(device)
        for item in tune:
            name, value = item.split("=")
            cz.cfgzip_set_tuning(self.ctx, name, int(value))
        self.parts = [cz.cfgzip_load_partition(self.ctx, p.c, p.V, p.r, p.K) for p in self.partitions]
        step_bytes = self.B * self.V * self.elem
        self.R = ring if ring else ring_steps(step_bytes, steps_hint)  # a short ring stays in L2: only for the figure labelled warm
        self.U = min(self.R, unique)
        # steps per CUDA graph: one pass over the ring; a short (L2-resident) ring is cycled 500 times per graph so
        # that the replay cost of a graph stays negligible there too
        self.G = self.R if not ring else 500 * self.R
        tile = -(-self.B // wl.B)
        tdt = torch.int16 if self.dtype == "bf16" else torch.float32
        self.host_logits = []
        self.pristine = []
        for u in range(self.U):
            z = np.tile(wl.logits(u), (tile, 1))[: self.B]
            self.host_logits.append(z)
            self.pristine.append(torch.from_numpy(z.view(np.int16) if self.dtype == "bf16" else z).cuda())
        self.host_cm = np.stack([self.w.class_masks(j) for j in range(self.R)])
        if allow_all:  # every class allowed (an unconstrained position of the grammar): the masks allow the whole vocabulary
            self.host_cm[:] = 0xFFFFFFFF
        self.cm = torch.from_numpy(self.host_cm.view(np.int32)).cuda()
        self.row_part_host = None if self.w.row_part is None else np.ascontiguousarray(self.w.row_part, dtype=np.int32)
        self.row_part = None if self.row_part_host is None else torch.from_numpy(self.row_part_host).cuda()
        self.row_part_arg = self.row_part
        if self.row_part is not None and kind == "fused":
            # the rows keep their grammars over the steps: group them by partition once, outside the steps
            cz.cfgzip_plan_rows(self.ctx, self.parts[0], self.row_part, self.B)
            self.row_part_arg = cz.ROWS_AS_PLANNED
        self.work = torch.empty((self.R, self.B, self.V), dtype=tdt, device="cuda")
        self.vm = torch.zeros((self.R, self.B, self.VW), dtype=torch.int32, device="cuda")
        self.am = torch.full((self.R, self.B), -9, dtype=torch.int32, device="cuda")
        self.rep = torch.full_like(self.am, -9)
        self.lse = torch.full((self.R, self.B), float("nan"), dtype=torch.float32, device="cuda")
        self.lpa = torch.full_like(self.lse, float("nan"))
        self.u = None
        if inv_temperature > 0:
            self.u = torch.from_numpy(np.stack([self.w.uniforms(j) for j in range(self.R)])).cuda()
        # automatic mode: the class masks come from the host (they are uploaded before the timed region), so the mode of
        # every step is chosen there with cfgzip_choose_mode, as a caller with a host-side grammar engine would
        self.step_modes = None
        if mode == "auto" and kind == "fused" and inv_temperature == 0:
            t0 = time.perf_counter()
            self.step_modes = [cz.cfgzip_choose_mode(self.ctx, self.parts[0], self.row_part_host, self.host_cm[j], self.KW, self.B,
                                                     cz.BF16 if self.dtype == "bf16" else cz.F32) for j in range(self.R)]
            self.choose_us_per_step = (time.perf_counter() - t0) / self.R * 1e6
        self.stream = torch.cuda.Stream()
        self.graph_obj = None
        self.launches_per_pass = 0
        self.pass_us_per_step = []
        self.restore()

    def close(self):
        self.graph_obj = None
        self.cz.cfgzip_destroy(self.ctx)

    def host_logits_of(self, j: int) -> np.ndarray:
        return self.host_logits[j % self.U]

    def restore(self, slots=None):
        """Refill working buffers with unmasked logits (outside any timed region)."""
        for j in (range(self.R) if slots is None else slots):
            self.work[j].copy_(self.pristine[j % self.U])
        self.torch.cuda.synchronize()

    def call(self, j: int, stream):
        cz = self.cz
        dt = cz.BF16 if self.dtype == "bf16" else cz.F32
        if self.kind == "floor":
            cz.cfgzip_rmw_floor(self.ctx, self.work[j], dt, self.V, self.B, self.V, stream)
        elif self.kind == "unfused":
            cz.cfgzip_expand_mask(self.ctx, self.parts[0], self.row_part, self.cm[j], self.KW, self.vm[j], self.VW,
                                  self.B, self.mode, stream)
            cz.cfgzip_mask_logits(self.ctx, self.work[j], dt, self.V, self.B, self.V, self.vm[j], self.VW, stream)
        elif self.u is not None:
            cz.cfgzip_masked_sample_filtered(
                self.ctx, self.parts[0], self.row_part_arg, self.cm[j], self.KW, self.work[j], dt, self.V, self.B,
                self.vm[j], self.VW, self.u[j], self.inv_temperature, self.top_k, self.top_p, self.am[j], self.rep[j],
                self.lpa[j], self.lse[j], self.mode, stream)
        else:
            cz.cfgzip_masked_logsoftmax_argmax(
                self.ctx, self.parts[0], self.row_part_arg, self.cm[j], self.KW, self.work[j], dt, self.V, self.B,
                self.vm[j], self.VW, self.am[j], self.rep[j], self.lpa[j], self.lse[j], None,
                self.mode if self.step_modes is None else self.step_modes[j], stream)

    def graph(self):
        """CUDA graph of one pass: steps 0..G-1 over the ring (captured once)."""
        if self.graph_obj is None:
            torch = self.torch
            g = torch.cuda.CUDAGraph()
            self.stream.wait_stream(torch.cuda.current_stream())
            before = self.cz.cfgzip_launch_count(self.ctx)
            with torch.cuda.stream(self.stream):
                with torch.cuda.graph(g, stream=self.stream):
                    for j in range(self.G):
                        self.call(j % self.R, self.stream)
            self.launches_per_pass = self.cz.cfgzip_launch_count(self.ctx) - before
            self.graph_obj = g
        return self.graph_obj

    def run_passes(self, passes: int, events=None) -> int:
        """Enqueue whole passes over the ring on self.stream; returns kernels launched."""
        g = self.graph()
        with self.torch.cuda.stream(self.stream):
            for _ in range(passes):
                g.replay()
                if events is not None:  # one event per pass, inside the timed region
                    ev = self.torch.cuda.Event(enable_timing=True)
                    ev.record(self.stream)
                    events.append(ev)
        return passes * self.launches_per_pass

    def timed(self, requested_steps: int, warmup: int, barrier=None, sampler: ClockSampler = None):
        """(seconds, timed steps, launches): whole passes over the ring, at least `requested_steps` steps and at least
        MIN_TIMED_SECONDS, after at least `warmup` (and at least 3) untimed steps; CUDA events on the launching stream."""
        torch = self.torch
        warm_passes = max(1, -(-max(warmup, 3) // self.G))
        self.run_passes(warm_passes)  # the first replay also uploads the graph
        self.stream.synchronize()
        # one more untimed pass, timed on its own, sizes the timed region
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record(self.stream)
        self.run_passes(1)
        p1.record(self.stream)
        self.stream.synchronize()
        n_steps = timed_steps_for(requested_steps, self.G, p0.elapsed_time(p1) * 1e-3)
        passes = n_steps // self.G
        if self.kind != "floor":
            self.restore()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        if barrier:
            barrier()
        if sampler:
            sampler.start()
        marks = []
        e0.record(self.stream)
        launched = self.run_passes(passes, marks)
        e1.record(self.stream)
        self.stream.synchronize()
        torch.cuda.synchronize()
        marks = [e0] + marks
        self.pass_us_per_step = [a.elapsed_time(b) * 1e3 / self.G for a, b in zip(marks, marks[1:])]
        if sampler:
            sampler.stop()
        if barrier:
            barrier()
        return e0.elapsed_time(e1) * 1e-3, n_steps, launched

    def execute_slots(self, slots, rows_sel, full_logits: int = 2) -> dict:
        """Run the steps of these ring slots once more on refilled buffers (untimed, no graph) and return the outputs
        of rows `rows_sel` as numpy arrays indexed [slot, row]; the masked logits of the first `full_logits` slots."""
        torch = self.torch
        slots = list(slots)
        idx = torch.tensor(slots, dtype=torch.long, device="cuda")
        rsel = torch.from_numpy(np.asarray(rows_sel, dtype=np.int64)).cuda()
        self.restore(slots)
        with torch.cuda.stream(self.stream):
            for j in slots:
                self.call(j, self.stream)
        self.stream.synchronize()

        def take(t):
            return t[idx][:, rsel].cpu().numpy()

        out = {"argmax": take(self.am), "rep": take(self.rep), "lse": take(self.lse), "logp_argmax": take(self.lpa),
               "vocab_mask": take(self.vm).view(np.uint32)}
        head = self.work[idx[:full_logits]][:, rsel].cpu().numpy()
        out["logits"] = head.view(np.uint16) if self.dtype == "bf16" else head
        return out

    def alg_bytes(self) -> int:
        if self.mode == self.cz.SPARSE and self.kind == "fused":
            return self.alg_bytes_sparse()
        return algorithmic_bytes(self.B, self.V, self.K, self.elem, len(self.parts))

    def alg_bytes_sparse(self) -> int:
        """Bytes one class-list step must move: write the whole row and its vocab mask, read the class masks, and per
        allowed token read its id from the class list (4 bytes) and its logit; mean over the first steps of the ring."""
        allowed_tokens = 0.0
        n = min(self.R, 8)
        for j in range(n):
            bits = synth.unpack_bits(self.host_cm[j], self.K)  # [B, K]
            for p, part in enumerate(self.partitions):
                sel = slice(None) if self.row_part_host is None else (self.row_part_host == p)
                allowed_tokens += float((bits[sel] * part.sizes[None, :]).sum())
        allowed_tokens /= n
        return int(self.B * (self.V * self.elem + 4 * self.VW + 4 * self.KW + 16) + allowed_tokens * (4 + self.elem))


def _measure(runner: StepRunner, min_steps: int = 300):
    """(us per step, steps timed, launches per step) of a secondary measurement: same protocol as the headline."""
    seconds, n, launched = runner.timed(min_steps, runner.G)
    return seconds / n * 1e6, n, launched / n


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


def _offline_grouping(cz, torch) -> dict:
    """cfgzip_group_tokens on a Llama-size vocabulary of synthetic signatures (2048 classes, 8-word rows), with the oracle's
    grouping of a sample beside it; the call allocates, synchronises and frees (an offline step), all inside the time."""
    V, K, W = 128256, 2048, 8
    part = synth.zipf_partition(V, K, 1.1, seed=3)
    rows = (synth.rng.u64(synth.rng.stream_key(8), K * W) % np.uint64(7)).astype(np.int32).reshape(K, W)
    rows[:, 1], rows[:, 2] = np.arange(K) // 7, np.arange(K) % 7
    sig = torch.from_numpy(np.ascontiguousarray(rows[part.c])).cuda()
    lens = torch.from_numpy((1 + synth.rng.u64(synth.rng.stream_key(9), V) % np.uint64(12)).astype(np.int32)).cuda()
    c = torch.empty(V, dtype=torch.int32, device="cuda"); r = torch.empty_like(c); k = torch.empty(1, dtype=torch.int32, device="cuda")
    off = torch.empty(V + 1, dtype=torch.int32, device="cuda"); tok = torch.empty_like(c)
    best = None
    for _ in range(5):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        cz.cfgzip_group_tokens(sig, W, lens, V, c, r, k, off, tok, torch.cuda.current_stream())
        dt_s = time.perf_counter() - t0
        best = dt_s if best is None else min(best, dt_s)
    ok = int(k.cpu()[0]) == K and bool((c.cpu().numpy() == _first_occurrence_ids(part.c)).all())
    return {"V": V, "classes": K, "row_words": W, "ms": best * 1e3, "tokens_per_s": V / best, "matches_partition": ok,
            "what": "grouping of equal signature rows into classes, representatives and class lists on the GPU, wall clock "
                    "of the whole call (allocation, 7 launches, synchronisation)"}


def _first_occurrence_ids(c: np.ndarray) -> np.ndarray:
    """Relabel class ids in the order of their lowest token id (bookkeeping for the check above)."""
    _, first, inverse = np.unique(c, return_index=True, return_inverse=True)
    rank = np.empty(len(first), dtype=np.int64)
    rank[np.argsort(first)] = np.arange(len(first))
    return rank[inverse]


def _multi_mask(cz, torch, device: int, B: int = 8, M: int = 16, steps: int = 200) -> dict:
    """cfgzip_multi_mask_logsoftmax_argmax: M class masks against each of B Llama-size rows (logits read once)."""
    w = synth.make_workload(2, B=B)
    part = w.partitions[0]
    ctx = cz.cfgzip_create(device)
    pid = cz.cfgzip_load_partition(ctx, part.c, w.V, part.r, w.K)
    z = torch.from_numpy(w.logits(0).view(np.int16)).cuda()
    cms = torch.from_numpy(synth.class_mask_bernoulli(w.K, B * M, 0.1, synth.rng.stream_key(77)).view(np.int32)).cuda()
    VW = (w.V + 31) // 32
    vm = torch.empty((B * M, VW), dtype=torch.int32, device="cuda")
    am = torch.empty(B * M, dtype=torch.int32, device="cuda"); rep = torch.empty_like(am)
    lse = torch.empty(B * M, dtype=torch.float32, device="cuda"); lpa = torch.empty_like(lse)
    st = torch.cuda.Stream()
    def run(n):
        with torch.cuda.stream(st):
            for _ in range(n):
                cz.cfgzip_multi_mask_logsoftmax_argmax(ctx, pid, cms, cms.shape[1], M, z, cz.BF16, w.V, B, vm, VW, am, rep, lpa, lse, st)
    run(20)
    st.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(st); run(steps); e1.record(st)
    st.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / steps
    cz.cfgzip_destroy(ctx)
    return {"B": B, "masks_per_row": M, "us_per_step": us, "row_masks_per_s": B * M / us * 1e6,
            "what": "V=128256 K=2048 bf16, one logits buffer (L2-resident: a latency figure, not an HBM one)"}


def _cpu_baseline(runner, budget_s: float = 12.0) -> dict:
    """The CPU oracle timed on steps of the same workload: with one thread per host core (rows split over a thread
    pool) and with a single thread, each for about half of `budget_s`."""
    import oracle
    threads = max(1, min(_host_threads(), runner.B))

    def timed(n_threads, budget):
        done, spent, j = 0, 0.0, 0
        while spent < budget:
            z = runner.host_logits_of(j).copy()
            t0 = time.perf_counter()
            oracle.decode_step(runner.partitions, runner.row_part_host, runner.host_cm[j % runner.R], z, threads=n_threads)
            spent += time.perf_counter() - t0
            done += 1
            j += 1
        return done, spent

    n_t, s_t = timed(threads, budget_s / 2)
    n_1, s_1 = timed(1, budget_s / 2)
    return {"value": n_t * runner.B / s_t, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "%d steps (%d rows) of the same workload, %d threads over rows" % (n_t, n_t * runner.B, threads),
            "single_thread": {"value": n_1 * runner.B / s_1, "unit": UNIT, "cores": 1,
                              "sample": "%d steps (%d rows) of the same workload, one thread" % (n_1, n_1 * runner.B)}}


# ----------------------------------------------------------------------------- arms

def run_own(args):
    import torch
    from paper_2605_29986_b200 import binding as cz

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CFGzip library has no CPU path")
    _, local_rank, _ = ranks.dist_env()
    torch.cuda.set_device(local_rank)
    os.environ.setdefault("NCCL_DEBUG", "INFO")       # the communicator's rank count shows in the log
    os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    rank, local_rank, world, dist = ranks.init_ranks("nccl", device=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()

    solo = rank == 0 and world == 1
    runner = StepRunner(cz, torch, local_rank, args.workload, B=args.batch, mode=args.mode, steps_hint=args.steps,
                        tune=args.tune, inv_temperature=args.sample_inv_temperature, top_k=args.top_k, top_p=args.top_p)
    props = torch.cuda.get_device_properties(local_rank)
    sampler = ClockSampler("GPU-" + str(props.uuid))
    seconds, timed_steps, launches = runner.timed(args.steps, args.warmup, barrier, sampler)
    e2e_steps = max(3, min(args.steps, args.e2e_steps))
    barrier()
    e2e_s, h2d, d2h = _e2e(runner, torch, e2e_steps)
    if dist is not None:
        seconds = ranks.max_over_ranks(seconds, dist, device="cuda")
        e2e_s = ranks.max_over_ranks(e2e_s, dist, device="cuda")
    peak, peak_src = _measured_peak()
    alg = runner.alg_bytes()
    us_per_step = seconds / timed_steps * 1e6
    # a dense step is two launches (streaming kernel + per-row finalize); the figure is per step
    achieved = alg / (seconds / timed_steps) / 1e9
    key = "cfg%d_B%d_%s" % (args.workload, runner.B, args.mode)
    traffic = None
    if key in NCU_TRAFFIC and NCU_TRAFFIC[key]["digest"] == _kernel_digest():
        traffic = NCU_TRAFFIC[key]["bytes_per_launch"]
    sampling = bool(args.sample_inv_temperature)
    line = {
        "metric": METRIC, "value": world * runner.B * timed_steps / seconds, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "timed_steps": timed_steps, "warmup": args.warmup, "ms_per_step": us_per_step * 1e-3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": runner.dtype,
        "data": "synthetic",
        "config": {
            "workload": "cfg%d %s: V=%d K=%d B=%d %s, fused expand+mask+lse+%s+rep, %s" % (
                args.workload, synth.CONFIGS[args.workload]["name"], runner.V, runner.K, runner.B, runner.dtype,
                "argmax" if not sampling else "sample(1/T=%g)" % args.sample_inv_temperature, args.mode),
            "rows_per_gpu": runner.B, "global_rows": world * runner.B,
            "l2": "inputs larger than L2: ring of %d working buffers (%.2f GB), refilled with unmasked logits before the "
                  "timed region" % (runner.R, runner.R * runner.B * runner.V * runner.elem / 1e9),
            "timed_region": "%d whole passes over the ring (%d steps, %.1f ms): at least the requested steps and at least "
                            "%.0f ms" % (timed_steps // runner.G, timed_steps, seconds * 1e3, MIN_TIMED_SECONDS * 1e3),
            "launch": "CUDA graph of one pass (%d steps) replayed, run untimed before the timed region; %.0f kernels per step" % (
                runner.G, launches / timed_steps),
            "inputs": "every row has its own class mask at every step; logits rows repeat every %d rows" % min(runner.B, 64),
            "parallelism": "rows sharded over %d GPU(s), no collective on the path" % world,
            "row_grouping": ("rows grouped by partition once before the steps (cfgzip_plan_rows), reused by every step"
                             if runner.row_part is not None else "one partition: rows grouped implicitly"),
        },
        "us_per_step": us_per_step,
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
                     "algorithmic_bytes_per_step": alg, "launches_per_step": launches / timed_steps,
                     "kernel": ("k_step_sparse" if args.mode == "sparse" else
                                "k_step_dense_pipe (+ %s)" % ("k_sample_rows" if sampling else "k_finalize_rows"))},
        "clocks": sampler.summary(),
        "paper_context": "paper reports no timing of this path; its speedups (up to two orders of magnitude in grammar-engine "
                         "latency, up to 7.5x end to end) are for 1x H100 + Xeon Gold 6430 x16 threads, precision unstated",
    }
    host_threads = max(1, min(_host_threads(), 16))
    if solo and not args.no_cpu_baseline and not sampling:
        # every step of the ring, every row (budget: a minute of oracle time)
        line["parity"] = check_slots(runner, range(runner.R), None, host_threads, budget_s=60.0)
        line["cpu_baseline"] = _cpu_baseline(runner)
    runner.close()
    if solo and not args.no_extras:
        def parity_of(r, steps=2, rows=32):
            if args.no_cpu_baseline:
                return None
            return check_slots(r, spread(r.R, steps), spread(r.B, rows), host_threads, budget_s=10.0)

        # the floor: the in-place read-modify-write kernel over the same ring, same graph protocol
        r0 = StepRunner(cz, torch, local_rank, args.workload, B=args.batch, steps_hint=args.steps, unique=2, tune=args.tune,
                        kind="floor")
        us0, _, _ = _measure(r0)
        r0.close()
        line["floor_us_per_step"] = us0
        line["roofline"]["floor"] = {"us_per_step": us0, "step_over_floor": us_per_step / us0,
                                     "what": "one launch per step that reads every logit of the batch and writes it back "
                                             "(sign flipped), same ring, same CUDA-graph protocol: the least a pass over "
                                             "these bytes costs here"}
        extras = []
        for B in (128, 256, 1024):
            r2 = StepRunner(cz, torch, local_rank, args.workload, B=B, mode=args.mode, steps_hint=8, unique=2, tune=args.tune)
            us2, n2, _ = _measure(r2)
            a2 = r2.alg_bytes() / us2 / 1e3
            entry = {"B": B, "us_per_step": us2, "rows_per_s": B / us2 * 1e6, "achieved_gbs": a2,
                     "frac_of_measured": a2 / peak, "ring": r2.R, "timed_steps": n2, "parity": parity_of(r2)}
            r2.close()
            rf = StepRunner(cz, torch, local_rank, args.workload, B=B, steps_hint=8, unique=2, tune=args.tune, kind="floor")
            entry["floor_us_per_step"] = _measure(rf)[0]
            rf.close()
            extras.append(entry)
        line["larger_batches"] = extras
        # the same masking through the two separate calls (expand, then mask; no normaliser, argmax or map):
        # the vocab mask is written and read back, so it moves more bytes for less work
        r3 = StepRunner(cz, torch, local_rank, args.workload, B=args.batch, mode=args.mode, steps_hint=256, unique=2,
                        tune=args.tune, kind="unfused")
        us3, _, l3 = _measure(r3)
        line["unfused_expand_then_mask"] = {"us_per_step": us3, "launches_per_step": l3}
        r3.close()
        # the sampling step (inverse CDF at the paper's temperature 0.2, one uniform number per row) on the same workload
        samp = []
        for B in (args.batch or synth.CONFIGS[args.workload]["B"], 1024):
            r6 = StepRunner(cz, torch, local_rank, args.workload, B=B, mode=args.mode, steps_hint=64, unique=2,
                            tune=args.tune, inv_temperature=5.0)
            us6, _, l6 = _measure(r6)
            samp.append({"B": B, "us_per_step": us6, "launches_per_step": l6,
                         "frac_of_measured": r6.alg_bytes() / us6 / 1e3 / peak})
            r6.close()
        line["sampling_step_T0.2"] = samp
        # the same sampling step restricted to the most probable tokens (top-k, top-p), at the paper's temperature
        filt = []
        for top_k, top_p in ((50, 1.0), (0, 0.9)):
            r8 = StepRunner(cz, torch, local_rank, args.workload, B=args.batch, mode=args.mode, steps_hint=64, unique=2,
                            tune=args.tune, inv_temperature=5.0, top_k=top_k, top_p=top_p)
            us8, _, l8 = _measure(r8)
            filt.append({"top_k": top_k, "top_p": top_p, "B": r8.B, "us_per_step": us8, "launches_per_step": l8})
            r8.close()
        # the same with masks that allow every class: far more tokens carry weight than the candidate list holds, and
        # the row is gone over a second time with a higher bar for the list
        r9 = StepRunner(cz, torch, local_rank, args.workload, B=args.batch, mode=args.mode, steps_hint=64, unique=2,
                        tune=args.tune, inv_temperature=5.0, top_k=50, top_p=0.9, allow_all=True)
        us9, _, l9 = _measure(r9)
        filt.append({"top_k": 50, "top_p": 0.9, "B": r9.B, "us_per_step": us9, "launches_per_step": l9,
                     "masks": "every class allowed"})
        r9.close()
        line["filtered_sampling_step_T0.2"] = filt
        line["offline_grouping"] = _offline_grouping(cz, torch)
        line["multi_mask_step"] = _multi_mask(cz, torch, local_rank)
        # the same step on two buffers that stay in the 126 MB L2: NOT an HBM figure, only the latency floor
        r5 = StepRunner(cz, torch, local_rank, args.workload, B=args.batch, mode=args.mode, steps_hint=2, unique=2,
                        tune=args.tune, ring=2)
        line["warm_l2_us_per_step"] = _measure(r5, 2000)[0]
        r5.close()
        # the five workloads at their own sizes (cfg2 is the headline above), same protocol
        five = []
        for cfg in sorted(synth.CONFIGS):
            r7 = StepRunner(cz, torch, local_rank, cfg, mode="dense", steps_hint=64, unique=2, tune=args.tune)
            us7, n7, l7 = _measure(r7)
            a7 = r7.alg_bytes() / us7 / 1e3
            all_steps = cfg in (1, 2)  # every step and row where the oracle takes seconds; a spread sample elsewhere
            par = None
            if not args.no_cpu_baseline:
                par = (check_slots(r7, range(r7.R), None, host_threads, budget_s=20.0) if all_steps else parity_of(r7))
            five.append({"workload": "cfg%d %s: V=%d K=%d B=%d %s, %d partition(s)" % (
                             cfg, synth.CONFIGS[cfg]["name"], r7.V, r7.K, r7.B, r7.dtype, len(r7.parts)),
                         "us_per_step": us7, "rows_per_s": r7.B / us7 * 1e6, "achieved_gbs": a7,
                         "frac_of_measured": a7 / peak, "launches_per_step": l7, "ring": r7.R, "timed_steps": n7,
                         "parity": par})
            r7.close()
        line["five_workloads_dense"] = five
        # sparse-mask stress workload (1-5 allowed classes per row): gather path, class-list scatter path, and the
        # library's own choice between them
        pair = {}
        for mode in ("dense", "sparse", "auto", "auto_on_device"):
            on_device = mode == "auto_on_device"
            r4 = StepRunner(cz, torch, local_rank, 5, mode="dense" if on_device else mode, steps_hint=4, unique=1,
                            tune=list(args.tune) + (["auto_min_mbytes=0"] if on_device else []))
            if on_device:
                r4.mode = cz.AUTO  # the GPU chooses, per batch of 8 rows (opt-in: one more launch)
            us4, _, _ = _measure(r4)
            pair[mode + "_us_per_step"] = us4
            if mode in ("dense", "sparse"):
                pair[mode + "_algorithmic_bytes"] = r4.alg_bytes()
                pair[mode + "_achieved_gbs_of_own_algorithmic_bytes"] = r4.alg_bytes() / us4 / 1e3
            if mode != "dense":
                pair[mode + "_parity"] = parity_of(r4)
            if mode == "auto":
                pair["auto_modes_chosen"] = sorted({{cz.DENSE: "dense", cz.SPARSE: "sparse"}[m] for m in r4.step_modes})
                pair["auto_choose_us_per_step_on_host"] = r4.choose_us_per_step
            r4.close()
        best = min(pair["dense_us_per_step"], pair["sparse_us_per_step"])
        pair["auto_vs_best"] = pair["auto_us_per_step"] / best
        pair["auto_on_device_vs_best"] = pair["auto_on_device_us_per_step"] / best
        pair["auto_what"] = ("auto: the mode of every step is chosen on the host from the class masks it is about to upload "
                             "(cfgzip_choose_mode, outside the timed region like the upload itself; its cost per step is given); "
                             "auto_on_device: CFGZIP_AUTO on device-resident masks with the opt-in knob, the class-list kernel "
                             "runs first and decides per batch of 8 rows, the gather kernel takes the rest (one more launch)")
        pair["workload"] = "cfg5 sparse-stress: V=128256 K=512 B=1024 f32"
        line["sparse_vs_dense"] = pair
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        if world > 1:
            time.sleep(0.5)  # let the other ranks' shutdown messages out first: the JSON line comes last
        print(json.dumps(line), flush=True)


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: each step is a bounded sample of the workload's rows."""
    rank, _, world = ranks.dist_env()
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


def main(argv=None):
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
    ap.add_argument("--top-k", type=int, default=0, help="with --sample-inv-temperature: keep the k most probable tokens")
    ap.add_argument("--top-p", type=float, default=1.0, help="with --sample-inv-temperature: keep the top-p nucleus")
    ap.add_argument("--no-extras", action="store_true", help="skip the larger-batch sweep")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args(argv)
    if args.steps < 1 or args.warmup < 0 or args.gpus < 1:
        ap.error("--steps and --gpus must be >= 1 and --warmup >= 0")
    if args.impl == "reference":
        run_reference(args)  # the CPU oracle: one process whatever --gpus says (under a launcher rank 0 alone runs it)
    elif ranks.need_spawn(args.gpus):
        # several GPUs asked for and no launcher in the environment: start one rank per GPU of this script
        sys.exit(ranks.spawn_ranks(os.path.abspath(__file__), args.gpus, sys.argv[1:] if argv is None else list(argv)))
    else:
        run_own(args)


if __name__ == "__main__":
    main()
