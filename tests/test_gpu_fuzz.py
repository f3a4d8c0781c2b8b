"""Seeded random shapes through the fused entry point: odd V, K and B, large class counts, padded strides,
both dtypes, dense and sparse. Every row (or a spread sample of rows when there are many) is compared with
the CPU oracle."""
import numpy as np
import pytest

import synth
from synth import rng
from paper_2605_29986_b200 import binding as cz
from _gpu_util import Ctx, compare_step, oracle_step, run_fused

pytestmark = pytest.mark.gpu


def _case(i):
    u = rng.u64(rng.stream_key(9001, i), 8)
    V = int(u[0] % np.uint64(300000)) + 1
    K = int(u[1] % np.uint64(min(V, 45000))) + 1
    B = int(u[2] % np.uint64(700)) + 1
    dtype = "bf16" if u[3] & np.uint64(1) else "f32"
    pad = int(u[4] % np.uint64(3)) * 8          # 0, 8 or 16 extra elements per row
    if u[7] % np.uint64(4):                     # three cases in four: rows on the 16-byte grid (fast kernels)
        pad += (-V) % 8
    dens = [0.002, 0.05, 0.3, 0.9][int(u[5] % np.uint64(4))]
    mode = cz.SPARSE if (u[6] % np.uint64(3)) == 0 else cz.DENSE
    return V, K, B, dtype, pad, dens, mode


@pytest.mark.parametrize("i", range(14))
def test_random_shape(i):
    V, K, B, dtype, pad, dens, mode = _case(i)
    part = synth.zipf_partition(V, K, 1.1, seed=i)
    cm = synth.class_mask_bernoulli(K, B, dens, rng.stream_key(9002, i))
    rows_u = min(B, 48)
    z = np.tile(synth.logits_normal(rows_u, V + pad, 2.0, dtype, (9003, i)), (-(-B // rows_u), 1))[:B]
    with Ctx([part]) as ctx:
        got = run_fused(ctx, None, cm, z, V, mode=mode, stride=V + pad)
        assert cz.cfgzip_poll_status(ctx.h)[1:] == (0, 0)
    rows = np.unique(np.linspace(0, B - 1, min(B, 40)).astype(np.int64))
    sub = {k: (v[rows] if v is not None else None) for k, v in got.items()}
    want = oracle_step([part], None, cm[rows], z[rows], V)
    compare_step(sub, want, V, "case %d: V=%d K=%d B=%d %s pad=%d dens=%g mode=%d" % (i, V, K, B, dtype, pad, dens, mode))
    assert np.array_equal(got["logits"][:, V:].view(np.uint8), z[:, V:].view(np.uint8))


@pytest.mark.parametrize("i", range(10))
def test_random_shape_sampling(i):
    # the sampling step over random shapes, temperatures and mask densities (aligned and unaligned rows)
    from test_gpu_sample import check_sample, run_sample
    u = rng.u64(rng.stream_key(7001, i), 8)
    V = int(u[0] % np.uint64(200000)) + 1
    K = int(u[1] % np.uint64(min(V, 20000))) + 1
    B = int(u[2] % np.uint64(300)) + 1
    dtype = "bf16" if u[3] & np.uint64(1) else "f32"
    pad = (-V) % 8 if (u[4] % np.uint64(4)) else 3
    inv_t = [0.5, 1.0, 5.0, 20.0][int(u[5] % np.uint64(4))]
    dens = [0.01, 0.1, 0.5][int(u[6] % np.uint64(3))]
    part = synth.zipf_partition(V, K, 1.1, seed=i)
    cm = synth.class_mask_bernoulli(K, B, dens, rng.stream_key(7002, i))
    cm[:, 0] |= 1
    rows_u = min(B, 32)
    z = np.tile(synth.logits_normal(rows_u, V + pad, 2.0, dtype, (7003, i)), (-(-B // rows_u), 1))[:B]
    uu = rng.uniform(rng.stream_key(7004, i), B).astype(np.float32)
    sel = np.unique(np.linspace(0, B - 1, min(B, 24)).astype(np.int64))
    with Ctx([part]) as ctx:
        got = run_sample(ctx, None, cm, z, V, uu, inv_t, stride=V + pad)
    sub = {k: (v[sel] if v is not None else None) for k, v in got.items()}
    near = check_sample(sub, [part], None, cm[sel], z[sel], V, uu[sel], inv_t, "case %d: V=%d K=%d B=%d %s" % (i, V, K, B, dtype))
    assert near <= 2
