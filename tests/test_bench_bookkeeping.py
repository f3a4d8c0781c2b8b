"""Host-side bookkeeping of bench.py, checked without a GPU: ring and timed-region sizes, the rule that the parity
leg only ever compares ring slots it has executed itself, and the launcher for several ranks."""
import json
import os
import subprocess
import sys

import numpy as np

import bench
import oracle
import synth
from paper_2605_29986_b200 import rows

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_ring_covers_a_gigabyte_and_the_requested_steps():
    step = 32 * 128256 * 2
    assert bench.ring_steps(step, 20) == -(-bench.RING_BYTES // step) == 131
    assert bench.ring_steps(step, 10000) == 1000
    assert bench.ring_steps(1024 * 128256 * 4, 10000) == bench.RING_MAX_BYTES // (1024 * 128256 * 4)
    assert bench.ring_steps(1 << 40, 5) == 1


def test_timed_region_is_whole_passes_and_long_enough():
    # 20 requested steps of 8.5 us on a ring of 131: one pass is 1.1 ms, so 18 passes are timed
    n = bench.timed_steps_for(20, 131, 131 * 8.5e-6)
    assert n % 131 == 0 and n * 8.5e-6 >= bench.MIN_TIMED_SECONDS and (n - 131) * 8.5e-6 < bench.MIN_TIMED_SECONDS
    assert bench.timed_steps_for(10000, 1000, 8.5e-3) == 10000     # long enough as requested
    assert bench.timed_steps_for(1001, 1000, 1.0) == 2000           # rounded up to whole passes
    assert bench.timed_steps_for(1, 4, 0.0) == 4


def test_spread_is_sorted_distinct_and_covers_both_ends():
    assert bench.spread(5, 10) == [0, 1, 2, 3, 4]
    s = bench.spread(1024, 32)
    assert s[0] == 0 and s[-1] == 1023 and s == sorted(set(s)) and len(s) == 32


class FakeRunner:
    """Stands in for the GPU ring: outputs exist only for slots that execute_slots was asked to run; every other slot
    holds the sentinel values the real output buffers are created with."""

    def __init__(self, R=6, B=5, corrupt_slot=None):
        self.w = synth.make_workload(2, B=B, V=3000, K=64)
        self.partitions, self.row_part_host = self.w.partitions, None
        self.R, self.B = R, B
        self.host_cm = np.stack([self.w.class_masks(j) for j in range(R)])
        self.executed = []
        self.corrupt_slot = corrupt_slot

    def host_logits_of(self, j):
        return self.w.logits(j % 2)

    def execute_slots(self, slots, rows_sel, full_logits=2):
        out = {k: [] for k in ("argmax", "rep", "lse", "logp_argmax", "vocab_mask", "logits")}
        for j in slots:
            self.executed.append(j)
            z = self.host_logits_of(j).copy()
            want = oracle.decode_step(self.partitions, None, self.host_cm[j], z)
            if j == self.corrupt_slot:
                want["argmax"] = want["argmax"].copy()
                want["argmax"][0] += 1
            for k in ("argmax", "rep", "vocab_mask"):
                out[k].append(want[k][rows_sel])
            out["lse"].append(want["lse"][rows_sel].astype(np.float32))
            out["logp_argmax"].append(want["logp_argmax"][rows_sel].astype(np.float32))
            out["logits"].append(z[rows_sel])
        out = {k: np.stack(v) for k, v in out.items()}
        out["logits"] = out["logits"][:full_logits]
        return out


def test_parity_leg_compares_only_slots_it_executed():
    r = FakeRunner()
    res = bench.check_slots(r, [0, 3, 5], [0, 2, 4])
    assert r.executed == [0, 3, 5]
    assert res["steps_checked"] == 3 and res["mismatching_steps"] == 0 and res["rows_per_step"] == 3
    assert res["of_ring_steps"] == 6 and res["of_rows"] == 5
    res = bench.check_slots(FakeRunner(), range(6))
    assert res["steps_checked"] == 6 and res["mismatching_steps"] == 0 and res["rows_per_step"] == 5


def test_parity_leg_counts_a_wrong_step():
    res = bench.check_slots(FakeRunner(corrupt_slot=3), range(6))
    assert res["steps_checked"] == 6 and res["mismatching_steps"] == 1


def test_gpus_flag_spawns_ranks_only_without_a_launcher():
    assert not rows.need_spawn(1, {})
    assert rows.need_spawn(8, {})
    assert not rows.need_spawn(8, {"RANK": "3", "WORLD_SIZE": "8", "LOCAL_RANK": "3"})
    assert rows.dist_env({"RANK": "3", "WORLD_SIZE": "8", "LOCAL_RANK": "3"}) == (3, 3, 8)
    assert rows.dist_env({}) == (0, 0, 1)
    cmd = rows.torchrun_command("bench.py", 4, ["--gpus", "4", "--steps", "20"], port=29123)
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node" in cmd and cmd[cmd.index("--nproc-per-node") + 1] == "4"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29123"
    assert cmd[-5:] == ["bench.py", "--gpus", "4", "--steps", "20"]


def test_launcher_starts_two_ranks_that_agree_on_the_slowest_time(tmp_path):
    # two CPU ranks (gloo) started by the same launcher the bench uses for --gpus N; a stub stands in for the GPU work
    out = tmp_path / "line.json"
    rc = rows.spawn_ranks(os.path.join(ROOT, "tests", "_stub_rank.py"), 2, [str(out)])
    assert rc == 0
    line = json.loads(out.read_text())
    assert line == {"n_gpus": 2, "seconds": 1.5, "rows": [[0, 4], [4, 7]]}
