"""cfgzip_step_noalloc: the fused step for callers that cannot allocate device memory.

Some users of the library sit inside another runtime's memory pool, or inside a region where
calling the CUDA allocator is forbidden, so they cannot create a context (which allocates
tables and scratch). The entry point tested here takes device-resident c and r from the
caller and keeps its only scratch in an array compiled into the library. The test drives it
through the C ABI twice in a row (the scratch array is shared and keeps the previous call's
contents) and compares every result with the context-based entry point and with the CPU oracle,
including a full 1024-row batch, one block per row, and class ids outside [0, K).

This file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

import synth
from synth import rng
from paper_2605_29986_b200 import binding as cz
from _gpu_util import Ctx, LOGP_TOL, compare_step, dev, dtype_code, host, oracle_step, run_fused

pytestmark = pytest.mark.gpu


def _noalloc(part, cm, z, V, stream=None):
    B = z.shape[0]
    VW = (V + 31) // 32
    d_c, d_r = dev(part.c), dev(part.r)
    d_z, d_cm = dev(z), dev(cm)
    d_vm = torch.full((B, VW), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    d_am = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    d_rep = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    d_lse = torch.full((B,), 123.0, dtype=torch.float32, device="cuda")
    d_lpa = torch.full((B,), 123.0, dtype=torch.float32, device="cuda")
    free_before = torch.cuda.mem_get_info()[0]
    cz.cfgzip_step_noalloc(d_c, V, d_r, part.K, d_cm, cm.shape[1], d_z, dtype_code(z), z.shape[1], B, d_vm, VW, d_am,
                           d_rep, d_lpa, d_lse, stream or torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_before  # the call took no device memory
    return dict(logits=host(d_z, z.dtype), vocab_mask=host(d_vm, np.uint32), argmax=d_am.cpu().numpy(),
                rep=d_rep.cpu().numpy(), lse=d_lse.cpu().numpy(), logp_argmax=d_lpa.cpu().numpy())


def _same(got, want, what):
    for key in ("vocab_mask", "logits", "argmax", "rep"):
        assert np.array_equal(got[key].view(np.uint8), want[key].view(np.uint8)), "%s: %s differs" % (what, key)
    for key in ("lse", "logp_argmax"):
        a, b = got[key].astype(np.float64), want[key].astype(np.float64)
        assert np.array_equal(np.isneginf(a), np.isneginf(b)), "%s: %s -inf pattern" % (what, key)
        fin = np.isfinite(b)
        assert not fin.any() or np.abs(a[fin] - b[fin]).max() <= LOGP_TOL, "%s: %s" % (what, key)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_noalloc_matches_the_context_entry_point_twice_in_a_row(dtype):
    V, K = 50003, 700                      # ragged vocabulary: rows off the 16-byte grid for bf16
    part = synth.zipf_partition(V, K, 1.1, seed=21)
    with Ctx([part]) as ctx:
        for call, B in enumerate((37, 5)):  # many rows (several blocks per row), then few (more blocks per row)
            cm = synth.class_mask_bernoulli(K, B, 0.15, rng.stream_key(77, call))
            cm[B // 2] = 0                  # one row with nothing allowed
            z = synth.logits_normal(B, V, 2.0, dtype, (78, call))
            want = run_fused(ctx, None, cm, z, V)
            _same(_noalloc(part, cm, z, V), want, "call %d" % call)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_noalloc_matches_the_oracle_twice_in_a_row(dtype):
    V, K = 50003, 700
    part = synth.zipf_partition(V, K, 1.1, seed=22)
    for call, B in enumerate((37, 5)):
        cm = synth.class_mask_bernoulli(K, B, 0.15, rng.stream_key(79, call))
        cm[B // 2] = 0
        z = synth.logits_normal(B, V, 2.0, dtype, (80, call))
        got = _noalloc(part, cm, z, V)
        got["logp_full"] = None
        compare_step(got, oracle_step([part], None, cm, z, V), V, "call %d" % call)


def test_noalloc_full_batch_one_block_per_row_against_the_oracle():
    # 1024 rows: the largest batch the built-in scratch takes, and so many rows that every row gets a single block
    # (the path that folds without tickets), with class masks that allow something in (almost) every row
    V, K, B = 9001, 130, 1024
    part = synth.zipf_partition(V, K, 1.1, seed=23)
    cm = synth.class_mask_bernoulli(K, B, 0.2, rng.stream_key(81))
    cm[17] = 0
    z = synth.logits_normal(B, V, 1.0, "bf16", (82,))
    for call in range(2):
        got = _noalloc(part, cm, z, V)
        got["logp_full"] = None
        compare_step(got, oracle_step([part], None, cm, z, V, threads=8), V, "call %d" % call)


def test_noalloc_treats_class_ids_out_of_range_as_disallowed():
    # the caller's device vector c is not validated: an id outside [0, K) must make its token disallowed and must not
    # index the class mask. The oracle sees the same thing as one more class (id K) that the mask never allows.
    V, K, B = 20000, 700, 9       # K = 700: bit 700 of the last class-mask word exists and stays 0
    part = synth.zipf_partition(V, K, 1.1, seed=24)
    cm = synth.class_mask_bernoulli(K, B, 0.3, rng.stream_key(83))
    z = synth.logits_normal(B, V, 2.0, "f32", (84,))
    bad = np.array([3, 777, 5000, 12345, 19999])
    bad = bad[~np.isin(bad, part.r)]              # keep every class's representative valid
    c_gpu = part.c.copy()
    c_gpu[bad] = np.array([K, -1, K + 1000, -2 ** 31, 2 ** 31 - 1])[: len(bad)]
    c_cpu = part.c.copy()
    c_cpu[bad] = K
    r_cpu = np.concatenate([part.r, bad[:1]]).astype(np.int32)
    cpu_part = synth.Partition(V=V, K=K + 1, c=c_cpu, r=r_cpu, sizes=np.bincount(c_cpu, minlength=K + 1))
    gpu_part = synth.Partition(V=V, K=K, c=c_gpu, r=part.r, sizes=part.sizes)
    z[:, bad] = 50.0                               # the tokens with bad ids would win every row if they were allowed
    got = _noalloc(gpu_part, cm, z, V)
    got["logp_full"] = None
    want = oracle_step([cpu_part], None, cm, z, V)
    compare_step(got, want, V, "bad class ids")
    assert not np.isin(got["argmax"], bad).any()


def test_noalloc_rejects_what_it_cannot_hold():
    lib = cz.load_library()
    part = synth.zipf_partition(1000, 10, 1.1, seed=1)
    d_c, d_r = dev(part.c), dev(part.r)
    B = 1025                                # one row more than the built-in scratch has tickets for
    d_cm = torch.zeros((B, 1), dtype=torch.int32, device="cuda")
    d_z = torch.zeros((B, 1000), dtype=torch.float32, device="cuda")
    d_am = torch.full((B,), -7, dtype=torch.int32, device="cuda")

    def call(b=B, c=d_c, k=10, cms=1, stride=1000):
        return lib.cfgzip_step_noalloc(cz._ptr(c), 1000, cz._ptr(d_r), k, cz._ptr(d_cm), cms, cz._ptr(d_z), cz.F32, stride, b,
                                       None, 0, cz._ptr(d_am), None, None, None, None)

    assert call() == cz.E_RANGE
    assert call(b=-1) == cz.E_ARG and call(c=None, b=4) == cz.E_ARG and call(b=4, cms=0) == cz.E_ARG
    assert call(b=4, stride=999) == cz.E_ARG and call(b=4, k=0) == cz.E_ARG
    torch.cuda.synchronize()
    assert d_am.cpu().numpy().tolist() == [-7] * B  # nothing ran
    assert call(b=1024) == cz.OK             # the largest batch it takes
    assert call(b=0) == cz.OK
    torch.cuda.synchronize()
    assert (d_am.cpu().numpy()[:1024] == -1).all()  # all-zero class masks: nothing allowed
