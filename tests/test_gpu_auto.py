"""CFGZIP_AUTO: the fused step that chooses, row by row and on the GPU, between the gather kernel and the
class-list kernel. The results must not depend on the choice, so every case is compared with the CPU oracle; the
cases mix groups that allow nearly everything with groups that allow a handful of classes, several partitions,
ragged vocabularies, rows with nothing allowed, and both thresholds' extremes (everything dense / everything lists).
"""
import numpy as np
import pytest

import synth
from synth import rng
from paper_2605_29986_b200 import binding as cz
from _gpu_util import Ctx, compare_step, oracle_step, run_fused

pytestmark = pytest.mark.gpu


def _mixed_masks(K, B, key, dense_rows):
    """Rows in `dense_rows` allow about 60 % of the classes, the others one to three classes."""
    cm = synth.class_mask_n_classes(K, B, 1, 3, rng.stream_key(key, 1))
    dense = synth.class_mask_bernoulli(K, B, 0.6, rng.stream_key(key, 2))
    cm[dense_rows] = dense[dense_rows]
    return cm


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("pct", [0, 250, 1000])
def test_auto_matches_the_oracle_whatever_it_chooses(pct, dtype):
    V, K, B = 20011 + 5, 300, 100                 # four row groups, the last one ragged
    part = synth.zipf_partition(V, K, 1.1, seed=31)
    dense_rows = np.r_[0:32, 64:100]              # groups 0, 2, 3 dense, group 1 sparse
    cm = _mixed_masks(K, B, 71, dense_rows)
    cm[5] = 0
    cm[40] = 0                                    # rows with nothing allowed in a dense and in a sparse group
    z = synth.logits_normal(B, V, 2.0, dtype, (72,))
    want = oracle_step([part], None, cm, z, V)
    with Ctx([part]) as ctx:
        cz.cfgzip_set_tuning(ctx.h, "auto_min_mbytes", 0)
        cz.cfgzip_set_tuning(ctx.h, "auto_sparse_permille", pct)
        before = cz.cfgzip_launch_count(ctx.h)
        for _ in range(2):
            compare_step(run_fused(ctx, None, cm, z, V, mode=cz.AUTO), want, V, "pct=%d" % pct)
        # streaming kernel + per-row kernel, and the class-list kernel in front whenever the choice is open
        assert cz.cfgzip_launch_count(ctx.h) - before == 2 * (3 if pct else 2)
        assert cz.cfgzip_poll_status(ctx.h) == (4, 0, 0)


def test_auto_with_mixed_partitions_and_a_kept_grouping():
    V, B = 30000, 90
    parts = [synth.zipf_partition(V, K, 1.1, seed=s) for s, K in enumerate((300, 256, 1024))]
    row_part = (np.arange(B) % 3).astype(np.int32)
    cm = synth.class_mask_n_classes(1024, B, 1, 2, rng.stream_key(73))
    cm &= np.uint32(0xFF)                          # classes 0..7 only: valid for every partition
    cm[:, 0] |= 1
    dense = synth.class_mask_bernoulli(256, B, 0.7, rng.stream_key(74))
    cm[row_part == 1, :8] = dense[row_part == 1]   # the rows of partition 1 allow most tokens, the others few
    z = synth.logits_normal(B, V, 1.0, "bf16", (75,))
    want = oracle_step(parts, row_part, cm, z, V)
    with Ctx(parts) as ctx:
        cz.cfgzip_set_tuning(ctx.h, "auto_min_mbytes", 0)
        cz.cfgzip_set_tuning(ctx.h, "auto_sparse_permille", 250)
        compare_step(run_fused(ctx, row_part, cm, z, V, mode=cz.AUTO), want, V)
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)


def test_auto_short_steps_are_dense_without_an_extra_launch():
    V, K, B = 20000, 300, 40
    part = synth.zipf_partition(V, K, 1.1, seed=32)
    cm = synth.class_mask_n_classes(K, B, 1, 3, rng.stream_key(76))
    z = synth.logits_normal(B, V, 2.0, "bf16", (77,))
    with Ctx([part]) as ctx:
        before = cz.cfgzip_launch_count(ctx.h)
        got = run_fused(ctx, None, cm, z, V, mode=cz.AUTO)
        assert cz.cfgzip_launch_count(ctx.h) - before == 2
    compare_step(got, oracle_step([part], None, cm, z, V), V)


def test_auto_on_the_sparse_stress_recipe_at_full_width():
    # 1 to 5 allowed classes of 512 over the Llama-size vocabulary, 96 rows: nearly every row stays with the class lists
    w = synth.make_workload(5, B=96)
    cm, z = w.class_masks(0), w.logits(0)
    with Ctx(w.partitions) as ctx:
        cz.cfgzip_set_tuning(ctx.h, "auto_min_mbytes", 0)
        got = run_fused(ctx, None, cm, z, w.V, mode=cz.AUTO)
        sparse = run_fused(ctx, None, cm, z, w.V, mode=cz.SPARSE)
    compare_step(got, oracle_step(w.partitions, None, cm, z, w.V), w.V)
    for key in ("vocab_mask", "logits", "argmax", "rep"):
        assert np.array_equal(got[key].view(np.uint8), sparse[key].view(np.uint8)), key
    assert np.abs(got["lse"] - sparse["lse"]).max() <= 1e-4   # rows with a large class allowed went to the gather kernel


def test_host_side_choice_and_the_host_buffer_step():
    # class masks born on the host (the grammar engine's side): the mode is chosen there, without a launch
    w = synth.make_workload(5, B=40, V=30000, K=128)
    part = w.partitions[0]
    sparse_cm, z = w.class_masks(0), w.logits(0)
    dense_cm = synth.class_mask_bernoulli(w.K, w.B, 0.5, rng.stream_key(78))
    lib = cz.load_library()
    with Ctx(w.partitions) as ctx:
        for cm, dtype in ((sparse_cm, cz.F32), (dense_cm, cz.F32), (sparse_cm, cz.BF16), (dense_cm, cz.BF16)):
            allowed = float((synth.unpack_bits(cm, w.K) * part.sizes[None, :]).sum()) / (w.B * w.V)
            want = cz.SPARSE if allowed * 1000 < (10 if dtype == cz.BF16 else 40) else cz.DENSE
            assert cz.cfgzip_choose_mode(ctx.h, ctx.ids[0], None, cm, cm.shape[1], w.B, dtype) == want
        assert cz.cfgzip_choose_mode(ctx.h, ctx.ids[0], None, dense_cm, dense_cm.shape[1], w.B, cz.F32) == cz.DENSE
        cz.cfgzip_set_tuning(ctx.h, "auto_sparse_permille", 1000)
        assert cz.cfgzip_choose_mode(ctx.h, ctx.ids[0], None, dense_cm, dense_cm.shape[1], w.B, cz.F32) == cz.SPARSE
        cz.cfgzip_set_tuning(ctx.h, "auto_sparse_permille", -1)
        assert lib.cfgzip_choose_mode(ctx.h, 7, None, dense_cm.ctypes.data, 4, w.B, cz.F32) == cz.E_RANGE
        assert lib.cfgzip_choose_mode(ctx.h, 0, None, None, 4, w.B, cz.F32) == cz.E_ARG
        assert lib.cfgzip_choose_mode(ctx.h, 0, None, dense_cm.ctypes.data, 3, w.B, cz.F32) == cz.E_ARG
        for cm in (sparse_cm, dense_cm):
            vm = np.empty((w.B, (w.V + 31) // 32), dtype=np.uint32); masked = np.empty_like(z)
            am = np.empty(w.B, dtype=np.int32); rep = np.empty(w.B, dtype=np.int32)
            lse = np.empty(w.B, dtype=np.float32); lpa = np.empty(w.B, dtype=np.float32)
            before = cz.cfgzip_launch_count(ctx.h)
            cz.cfgzip_decode_step_host(ctx.h, ctx.ids[0], None, cm, cm.shape[1], z, cz.F32, w.B, masked, vm, am, rep, lpa, lse,
                                       cz.AUTO)
            assert cz.cfgzip_launch_count(ctx.h) - before == (1 if cm is sparse_cm else 2)   # class-list kernel alone / gather + per-row
            got = dict(logits=masked, vocab_mask=vm, argmax=am, rep=rep, lse=lse, logp_argmax=lpa)
            compare_step(got, oracle_step(w.partitions, None, cm, z, w.V), w.V)
