"""The five workloads at their full sizes, through the fused entry point in the launch shape the bench uses.

Inputs follow the workload recipes (unique logits rows are generated for up to 64 rows and tiled to
the batch, and repeat every 16 steps; every row has its own class mask at every step). Every decode
step of the two small workloads and ten steps spread over the run of the others are covered. All rows
are compared with the CPU oracle where that takes seconds; for the largest batch a spread sample of
rows is compared and the remaining rows are checked by properties that hold at any size (popcount of the vocab mask = summed sizes of the
allowed classes, -inf count of the masked logits, the chosen token is allowed and maps to its
representative) and, for the sparse stress workload, by bit-equality of the dense and sparse paths.
"""
import numpy as np
import pytest
import torch

import synth
from paper_2605_29986_b200 import binding as cz
from _gpu_util import Ctx, compare_step, oracle_step, run_fused

pytestmark = pytest.mark.gpu

# rows of a step that are compared with the oracle one by one (the rest: properties that hold at any size)
ORACLE_ROWS = {1: 1, 2: 32, 3: 128, 4: 256, 5: 64}
# decode steps covered: every step of the two small workloads, ten spread over the run of the others
STEPS = {1: list(range(100)), 2: list(range(1000)),
         3: [int(x) for x in np.linspace(0, 499, 10)], 4: [int(x) for x in np.linspace(0, 199, 10)],
         5: [int(x) for x in np.linspace(0, 199, 10)]}
# the logits of step s are those of step s mod FRESH_LOGITS (generating them costs far more than the step itself)
FRESH_LOGITS = {1: 100, 2: 16, 3: 16, 4: 16, 5: 16}
_logits_cache = {}


def _inputs(config, step):
    spec = synth.CONFIGS[config]
    B = spec["B"]
    fresh = step % FRESH_LOGITS[config]
    if ("w", config) not in _logits_cache:
        _logits_cache.clear()
        _logits_cache[("w", config)] = synth.make_workload(config, B=min(B, 64))   # unique logits rows
    wu = _logits_cache[("w", config)]
    if fresh not in _logits_cache:
        _logits_cache[fresh] = wu.logits(fresh)
    z = np.tile(_logits_cache[fresh], (-(-B // wu.B), 1))[:B]
    wf = _workload(config)                                 # class masks (and partitions) for every row
    cm = wf.class_masks(step)
    row_part = None if wf.row_part is None else wf.row_part
    return wf, row_part, cm, z


_workloads = {}


def _workload(config):
    if config not in _workloads:
        _workloads.clear()
        _workloads[config] = synth.make_workload(config)
    return _workloads[config]


def _popcount_rows(words):
    return np.unpackbits(np.ascontiguousarray(words).view(np.uint8), axis=-1).sum(axis=-1)


def _properties(w, row_part, cm, got, V):
    B = cm.shape[0]
    pc = _popcount_rows(got["vocab_mask"])
    neg = (got["logits"].view(np.uint16 if got["logits"].dtype == np.uint16 else np.uint32)
           == (0xFF80 if got["logits"].dtype == np.uint16 else 0xFF800000)).sum(axis=1)
    for b in range(B):
        p = w.partitions[0 if row_part is None else int(row_part[b])]
        allowed = synth.unpack_bits(cm[b:b + 1], p.K)[0]
        assert pc[b] == int(p.sizes[allowed].sum()), "row %d popcount" % b
        assert neg[b] >= V - pc[b]
        t = int(got["argmax"][b])
        if pc[b] == 0:
            assert t == -1 and got["rep"][b] == -1
        else:
            assert allowed[p.c[t]] and got["rep"][b] == p.r[p.c[t]]
            assert got["logp_argmax"][b] <= 1e-6


@pytest.mark.parametrize("config", [1, 2, 3, 4, 5])
def test_full_size_workload(config):
    spec = synth.CONFIGS[config]
    V, B = spec["V"], spec["B"]
    w = _workload(config)
    with Ctx(w.partitions) as ctx:
        for n, step in enumerate(STEPS[config]):
            _, row_part, cm, z = _inputs(config, step)
            got = run_fused(ctx, row_part, cm, z, V, mode=cz.DENSE)
            if config == 5:
                sparse = run_fused(ctx, row_part, cm, z, V, mode=cz.SPARSE)
                for key in ("vocab_mask", "logits", "argmax", "rep"):
                    assert np.array_equal(got[key].view(np.uint8), sparse[key].view(np.uint8)), key
                assert np.abs(got["lse"] - sparse["lse"]).max() <= 1e-4
            if n % 10 == 0 or len(STEPS[config]) <= 10:
                _properties(w, row_part, cm, got, V)
            rows = np.unique(np.linspace(0, B - 1, ORACLE_ROWS[config]).astype(np.int64))
            sub = {k: (v[rows] if v is not None else None) for k, v in got.items()}
            want = oracle_step(w.partitions, None if row_part is None else row_part[rows], cm[rows], z[rows], V)
            compare_step(sub, want, V, "config %d step %d" % (config, step))
        assert cz.cfgzip_poll_status(ctx.h)[1:] == (0, 0)


@pytest.mark.parametrize("B", [256, 1024])
def test_llama_size_large_batches_three_stage_launch(B):
    # the launch shapes the bench's larger batches use: two stages per warp at 256 rows, three at 1024 rows with the
    # class-mask staging area laid over the first rings
    plan = cz.cfgzip_plan_query(148, 232448, 128256, 2048, B, cz.BF16)
    assert plan["kind"] == 2 and plan["depth"] == (3 if B >= 1024 else 2)
    wu = synth.make_workload(2, B=64)
    wf = synth.make_workload(2, B=B)
    z = np.tile(wu.logits(3), (B // 64, 1))
    cm = wf.class_masks(3)
    with Ctx(wf.partitions) as ctx:
        got = run_fused(ctx, None, cm, z, wf.V, mode=cz.DENSE)
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)
    _properties(wf, None, cm, got, wf.V)
    rows = np.unique(np.linspace(0, B - 1, 96).astype(np.int64))
    sub = {k: (v[rows] if v is not None else None) for k, v in got.items()}
    compare_step(sub, oracle_step(wf.partitions, None, cm[rows], z[rows], wf.V), wf.V, "B=%d" % B)


def test_heavy_tail_workload_with_kept_row_grouping():
    # the bench groups the rows of the mixed batch once (cfgzip_plan_rows) and reuses the grouping at every step
    w, row_part, cm, z = _inputs(4, 2)
    V, B = w.V, cm.shape[0]
    VW = (V + 31) // 32
    from _gpu_util import dev, host
    with Ctx(w.partitions) as ctx:
        d_rp = dev(row_part)
        cz.cfgzip_plan_rows(ctx.h, ctx.ids[0], d_rp, B)
        d_z, d_cm = dev(z), dev(cm)
        d_vm = torch.zeros((B, VW), dtype=torch.int32, device="cuda")
        d_am = torch.zeros(B, dtype=torch.int32, device="cuda")
        d_rep = torch.zeros_like(d_am)
        d_lse = torch.zeros(B, dtype=torch.float32, device="cuda")
        d_lpa = torch.zeros_like(d_lse)
        cz.cfgzip_masked_logsoftmax_argmax(ctx.h, ctx.ids[0], cz.ROWS_AS_PLANNED, d_cm, cm.shape[1], d_z, cz.BF16, V, B, d_vm,
                                           VW, d_am, d_rep, d_lpa, d_lse, None, cz.DENSE)
        torch.cuda.synchronize()
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)
        got = dict(logits=host(d_z, z.dtype), vocab_mask=host(d_vm, np.uint32), argmax=d_am.cpu().numpy(),
                   rep=d_rep.cpu().numpy(), lse=d_lse.cpu().numpy(), logp_argmax=d_lpa.cpu().numpy(), logp_full=None)
    _properties(w, row_part, cm, got, V)
    rows = np.unique(np.linspace(0, B - 1, 48).astype(np.int64))
    sub = {k: (v[rows] if v is not None else None) for k, v in got.items()}
    compare_step(sub, oracle_step(w.partitions, row_part[rows], cm[rows], z[rows], V), V, "kept grouping")
