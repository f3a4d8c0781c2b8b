"""The bf16 streaming kernel with two octets (16 tokens, 32 bytes) per lane and row, forced on shapes where the
library would not choose it by itself, against the CPU oracle; and the kernel's error path for a copy that is
reported as never arrived.

Shapes put the end of the vocabulary at every place inside a 512-token chunk that the kernel treats differently
(first or second box of the chunk, first or second octet of a lane, a ragged octet, none), rows on and off the
32-byte grid, row batches with fewer than 8 rows, several row groups, and mixed partitions (one copy per row
instead of tiled copies).
"""
import numpy as np
import pytest
import torch

import synth
from synth import rng
from paper_2605_29986_b200 import binding as cz
from _gpu_util import Ctx, compare_step, oracle_step, run_fused
from test_gpu_sample import check_sample, run_sample

pytestmark = pytest.mark.gpu


def _mask(K, B, p, *ids):
    return synth.class_mask_bernoulli(K, B, p, rng.stream_key(5151, *ids))


def _two_octets(ctx, **more):
    cz.cfgzip_set_tuning(ctx.h, "lane_octets", 2)
    for name, value in more.items():
        cz.cfgzip_set_tuning(ctx.h, name, value)


# V: ends inside the first box (200), exactly one box (256), one octet into the second box (264), odd octet count
# (504), a whole chunk (512), a chunk and a ragged octet (515), several chunks with every kind of end
@pytest.mark.parametrize("V", [8, 16, 24, 200, 256, 264, 504, 512, 515, 1000, 1031, 4096, 4099, 20011 + 5])
def test_two_octets_per_lane_tiny_and_ragged(V):
    K = min(V, 37)
    part = synth.zipf_partition(V, K, 1.1, seed=V + 7)
    stride = -(-V // 8) * 8                       # rows on the 16-byte grid; on the 32-byte grid only if V % 16 < 9
    for B in (1, 5, 33):
        cm = _mask(K, B, 0.5, V, B)
        z = synth.logits_normal(B, stride, 2.0, "bf16", (61, V, B))
        want = oracle_step([part], None, cm, z, V)
        for knobs in (dict(), dict(tensor_map=0), dict(pipe_warps=4, pipe_depth=3)):
            with Ctx([part]) as ctx:
                _two_octets(ctx, **knobs)
                got = run_fused(ctx, None, cm, z, V, stride=stride)
                assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)
            compare_step(got, want, V, "V=%d B=%d %r" % (V, B, knobs))
            assert np.array_equal(got["logits"][:, V:].view(np.uint8), z[:, V:].view(np.uint8))  # padding untouched


@pytest.mark.parametrize("stride_pad", [0, 8, 16])
def test_two_octets_per_lane_several_groups_and_chunks(stride_pad):
    # 70 rows = two full row groups and a ragged third with a 6-row batch; rows 32-byte aligned only for pad 0 and 16
    V, K, B = 50000, 700, 70
    stride = V + stride_pad
    part = synth.zipf_partition(V, K, 1.1, seed=8)
    cm = _mask(K, B, 0.1, stride_pad)
    z = synth.logits_normal(B, stride, 2.0, "bf16", (62,))
    want = oracle_step([part], None, cm, z, V)
    with Ctx([part]) as ctx:
        _two_octets(ctx)
        for _ in range(2):
            got = run_fused(ctx, None, cm, z, V, stride=stride, vm_stride=(V + 31) // 32 + 1)
            compare_step(got, want, V)
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)


def test_two_octets_per_lane_mixed_partitions():
    V, B = 20011 + 5, 70
    parts = [synth.zipf_partition(V, K, 1.1, seed=s) for s, K in enumerate((300, 256, 1024))]
    row_part = (rng.u64(rng.stream_key(2), B) % np.uint64(3)).astype(np.int32)
    cm = _mask(1024, B, 0.2, 9)
    z = synth.logits_normal(B, V, 2.0, "bf16", (63,))
    with Ctx(parts) as ctx:
        _two_octets(ctx)
        got = run_fused(ctx, row_part, cm, z, V)
    compare_step(got, oracle_step(parts, row_part, cm, z, V), V)


def test_two_octets_per_lane_sampling_step():
    V, K, B = 30000 + 24, 300, 40
    part = synth.zipf_partition(V, K, 1.1, seed=9)
    cm = _mask(K, B, 0.2, 11)
    z = synth.logits_normal(B, V, 2.0, "bf16", (64,))
    u = rng.uniform(rng.stream_key(65), B).astype(np.float32)
    with Ctx([part]) as ctx:
        _two_octets(ctx)
        got = run_sample(ctx, None, cm, z, V, u, 5.0)
        near = check_sample(got, [part], None, cm, z, V, u, 5.0)
    assert near <= 2


@pytest.mark.parametrize("dtype,octets", [("bf16", 1), ("bf16", 2), ("f32", 0)])
def test_a_copy_reported_as_never_arrived_surfaces_as_an_error(dtype, octets):
    # The streaming kernel waits for its asynchronous copies with a bounded wait; when one runs out the warp flags
    # it, waits (bounded again) for its other copies in flight and leaves, and cfgzip_poll_status reports
    # CFGZIP_E_CUDA. The test hook makes every warp treat its first, completed, wait as run out, so the whole
    # path runs while every copy has in fact landed: nothing hangs and no memory is left in flight.
    V, K, B = 40000, 300, 40
    part = synth.zipf_partition(V, K, 1.1, seed=10)
    cm = _mask(K, B, 0.2, 12)
    z = synth.logits_normal(B, V, 2.0, dtype, (66,))
    want = oracle_step([part], None, cm, z, V)
    lib = cz.load_library()
    with Ctx([part]) as ctx:
        if octets:
            cz.cfgzip_set_tuning(ctx.h, "lane_octets", octets)
        compare_step(run_fused(ctx, None, cm, z, V), want, V)          # a normal step first
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)
        cz.cfgzip_set_tuning(ctx.h, "test_expire_waits", 1)
        run_fused(ctx, None, cm, z, V)                                   # results of this call are undefined
        assert lib.cfgzip_poll_status(ctx.h, None, None, None, None) == cz.E_CUDA
        cz.cfgzip_set_tuning(ctx.h, "test_expire_waits", 0)
        compare_step(run_fused(ctx, None, cm, z, V), want, V)          # the context stays usable
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("fold", [1, 2])
def test_results_written_by_the_streaming_kernel_itself(fold, dtype):
    # "fold" = 1: the last block of a row group to finish folds the group's states and writes the results (one launch
    # per step); 2: the warps of a block merge their states in shared memory first and a second launch finishes the
    # rows. Both are alternatives to the default (per-warp states, second launch) and must give the same step.
    for V, K, B, parts in ((515, 37, 1, 1), (4099, 130, 33, 1), (50000, 700, 70, 1), (20011 + 5, 300, 70, 3)):
        ps = [synth.zipf_partition(V, K, 1.1, seed=40 + s) for s in range(parts)]
        row_part = None if parts == 1 else (rng.u64(rng.stream_key(3), B) % np.uint64(parts)).astype(np.int32)
        cm = _mask(K, B, 0.2, V, fold)
        if B > 2:
            cm[B // 2] = 0                                   # a row with nothing allowed
        z = synth.logits_normal(B, -(-V // 8) * 8, 2.0, dtype, (67, V))
        want = oracle_step(ps, row_part, cm, z, V)
        with Ctx(ps) as ctx:
            cz.cfgzip_set_tuning(ctx.h, "fold", fold)
            before = cz.cfgzip_launch_count(ctx.h)
            for _ in range(2):                               # twice: the tickets are left ready for the next launch
                compare_step(run_fused(ctx, row_part, cm, z, V, stride=z.shape[1]), want, V, "V=%d B=%d" % (V, B))
            launches = cz.cfgzip_launch_count(ctx.h) - before
            assert launches == 2 * ((1 if fold == 1 else 2) + (1 if parts > 1 else 0))
            assert cz.cfgzip_poll_status(ctx.h)[1:] == (0, 0)
