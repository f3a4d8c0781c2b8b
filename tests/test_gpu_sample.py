"""GPU parity of the sampling step (cfgzip_masked_sample) against the CPU oracle.

Vocab masks, masked logits and representative ids are compared bit for bit. The sampled token is an
integer decided by floating-point sums (fp32 on the GPU, fp64 in the oracle): it must equal the
oracle's wherever the row's uniform number lies further than CDF_TOL from every boundary of the
oracle's cumulative distribution; closer than that, either neighbour of the boundary is a valid
draw, so the test checks that the GPU's token is allowed, has positive probability and that u lies
within CDF_TOL of that token's interval of the oracle's CDF. lse and logp_token: 1e-4 absolute.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from synth import rng
from paper_2605_29986_b200 import binding as cz
from _gpu_util import Ctx, assert_close_log, dev, dtype_code, host

pytestmark = pytest.mark.gpu

CDF_TOL = 2e-5


def run_sample(ctx, row_part, cm, z, V, u, inv_t, stride=None, mode=cz.DENSE, want_vm=True):
    B = z.shape[0]
    stride = stride or z.shape[1]
    VW = (V + 31) // 32
    d_z, d_cm, d_u = dev(z), dev(cm), dev(np.asarray(u, dtype=np.float32))
    d_rp = None if row_part is None else dev(np.asarray(row_part, dtype=np.int32))
    d_vm = torch.full((B, VW), 0x5A5A5A5A, dtype=torch.int32, device="cuda") if want_vm else None
    d_tok = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    d_rep = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    d_lse = torch.full((B,), 123.0, dtype=torch.float32, device="cuda")
    d_lpt = torch.full((B,), 123.0, dtype=torch.float32, device="cuda")
    cz.cfgzip_masked_sample(ctx.h, ctx.ids[0], d_rp, d_cm, cm.shape[1], d_z, dtype_code(z), stride, B, d_vm, VW, d_u,
                            inv_t, d_tok, d_rep, d_lpt, d_lse, mode, torch.cuda.current_stream())
    torch.cuda.synchronize()
    return dict(logits=host(d_z, z.dtype), vocab_mask=None if d_vm is None else host(d_vm, np.uint32),
                token=d_tok.cpu().numpy(), rep=d_rep.cpu().numpy(), lse=d_lse.cpu().numpy(),
                logp_token=d_lpt.cpu().numpy())


def check_sample(got, partitions, row_part, cm, z, V, u, inv_t, what=""):
    """Compare one GPU sampling step with the oracle; returns the number of rows decided on a boundary."""
    zc = np.ascontiguousarray(z[:, :V]).copy()
    u64 = np.asarray(u, dtype=np.float32).astype(np.float64)
    want = oracle.sample_step(partitions, row_part, cm, zc, float(inv_t), u64, want_cdf=True, threads=8)
    if got["vocab_mask"] is not None:
        assert np.array_equal(got["vocab_mask"], want["vocab_mask"]), what + " vocab mask"
    assert np.array_equal(got["logits"][:, :V].view(np.uint8), zc.view(np.uint8)), what + " masked logits"
    assert_close_log(got["lse"], want["lse"], what + " lse")
    near = 0
    for b in range(z.shape[0]):
        t, tw = int(got["token"][b]), int(want["token"][b])
        part = partitions[0 if row_part is None else int(row_part[b])]
        if t != tw:
            # only a boundary case may differ: t allowed, positive probability, u within CDF_TOL of its CDF interval
            assert t >= 0 and tw >= 0, (what, b, t, tw)
            cdf = want["cdf"][b]
            hi = cdf[t]
            lo = cdf[t - 1] if t > 0 else 0.0
            assert (int(want["vocab_mask"][b, t // 32]) >> (t % 32)) & 1 == 1, (what, b, t)
            assert hi > lo, (what, b, t, "zero-probability token drawn")
            assert lo - CDF_TOL <= u64[b] <= hi + CDF_TOL, (what, b, t, tw, lo, hi, u64[b])
            near += 1
            # the oracle's own log-probability of the token the GPU drew: z_t / T - lse
            zt = float(rng.bf16_bits_to_f32(zc[b, t:t + 1])[0]) if zc.dtype == np.uint16 else float(zc[b, t])
            want_lpt = zt * float(inv_t) - want["lse"][b]
            assert abs(got["logp_token"][b] - want_lpt) <= 1e-4, (what, b, got["logp_token"][b], want_lpt)
        else:
            if np.isneginf(want["logp_token"][b]):
                assert np.isneginf(got["logp_token"][b]), (what, b)
            else:
                assert abs(got["logp_token"][b] - want["logp_token"][b]) <= 1e-4, (what, b, got["logp_token"][b], want["logp_token"][b])
        want_rep = -1 if t < 0 else int(part.r[part.c[t]])
        assert int(got["rep"][b]) == want_rep, (what, b)
    return near


TINY = [(1, 1), (7, 3), (31, 2), (33, 32), (63, 33), (65, 64), (255, 9), (256, 16), (257, 40), (1000, 37), (4099, 130)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,K", TINY)
def test_sample_tiny_shapes(V, K, dtype):
    part = synth.zipf_partition(V, K, 1.1, seed=V)
    near = rows = 0
    with Ctx([part]) as ctx:
        for B, inv_t in ((1, 1.0), (5, 5.0), (33, 0.5)):
            cm = synth.class_mask_bernoulli(K, B, 0.5, rng.stream_key(31, V, B))
            cm[:, 0] |= 1  # at least one class allowed
            z = synth.logits_normal(B, V, 2.0, dtype, (32, V, B))
            u = rng.uniform(rng.stream_key(33, V, B), B).astype(np.float32)
            got = run_sample(ctx, None, cm, z, V, u, inv_t)
            near += check_sample(got, [part], None, cm, z, V, u, inv_t, "V=%d K=%d B=%d" % (V, K, B))
            rows += B
    assert near <= max(1, rows // 10)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sample_unaligned_rows_take_the_per_row_path(dtype):
    V, K, B, stride = 3001, 77, 9, 3003
    part = synth.zipf_partition(V, K, 1.1, seed=4)
    cm = synth.class_mask_bernoulli(K, B, 0.3, rng.stream_key(41))
    z = synth.logits_normal(B, stride, 1.0, dtype, (42,))
    u = rng.uniform(rng.stream_key(43), B).astype(np.float32)
    with Ctx([part]) as ctx:
        got = run_sample(ctx, None, cm, z, V, u, 5.0, stride=stride)
        check_sample(got, [part], None, cm, z, V, u, 5.0)
        assert np.array_equal(got["logits"][:, V:].view(np.uint8), z[:, V:].view(np.uint8))  # padding untouched


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sample_several_groups_and_vocabulary_tiles(dtype):
    # several row groups, many chunks per warp slot, a ragged end (V % 8 != 0) and padded rows
    V, K, B = 70003, 900, 75
    stride = 70008
    part = synth.zipf_partition(V, K, 1.1, seed=5)
    cm = synth.class_mask_bernoulli(K, B, 0.1, rng.stream_key(51))
    z = synth.logits_normal(B, stride, 2.0, dtype, (52,))
    near = 0
    with Ctx([part]) as ctx:
        for trial, inv_t in enumerate((1.0, 5.0)):
            u = rng.uniform(rng.stream_key(53, trial), B).astype(np.float32)
            got = run_sample(ctx, None, cm, z, V, u, inv_t, stride=stride)
            near += check_sample(got, [part], None, cm, z, V, u, inv_t, "trial %d" % trial)
    assert near <= 4


def test_sample_mixed_partitions():
    w = synth.make_workload(4, B=70, V=30000, K=700)
    cm, z, u = w.class_masks(0), w.logits(0), w.uniforms(0)
    with Ctx(w.partitions) as ctx:
        got = run_sample(ctx, w.row_part, cm, z, w.V, u, 5.0)
        near = check_sample(got, w.partitions, w.row_part, cm, z, w.V, u, 5.0)
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)
    assert near <= 2


def test_sample_edge_rows_and_extreme_uniforms():
    V, K, B = 5000, 64, 8
    part = synth.zipf_partition(V, K, 1.1, seed=6)
    cm = synth.class_mask_bernoulli(K, B, 0.3, rng.stream_key(61))
    cm[0] = 0                       # nothing allowed
    z = synth.logits_normal(B, V, 1.0, "f32", (62,))
    allowed1 = synth.unpack_bits(oracle.expand_mask(part.c, K, cm[1:2]), V)[0]
    z[1, allowed1] = -np.inf        # allowed logits all -inf
    u = np.array([0.5, 0.5, 0.0, np.float32(1.0) - np.float32(2.0 ** -24), 0.25, 0.5, 0.75, 0.999], dtype=np.float32)
    with Ctx([part]) as ctx:
        got = run_sample(ctx, None, cm, z, V, u, 2.0)
        check_sample(got, [part], None, cm, z, V, u, 2.0)
        assert got["token"][0] == -1 and got["rep"][0] == -1 and np.isneginf(got["lse"][0])
        assert got["token"][1] == np.flatnonzero(allowed1)[0] and np.isneginf(got["logp_token"][1])
        assert cz.cfgzip_poll_status(ctx.h)[0] == 1  # one row with nothing allowed
        # the same call again gives the same answer (fixed summation order)
        again = run_sample(ctx, None, cm, z, V, u, 2.0)
        for k in ("token", "rep", "lse", "logp_token"):
            assert np.array_equal(got[k], again[k], equal_nan=True), k


def test_sample_cold_distribution_is_the_greedy_choice_and_t1_matches_the_greedy_lse():
    w = synth.make_workload(2, B=40, V=20000, K=300)
    cm, z = w.class_masks(1), w.logits(1)
    u = np.minimum(w.uniforms(1), np.float32(0.99))
    zc = z.copy()
    want = oracle.decode_step(w.partitions, None, cm, zc)
    with Ctx(w.partitions) as ctx:
        cold = run_sample(ctx, None, cm, z, w.V, u, 200.0)
        t1 = run_sample(ctx, None, cm, z, w.V, u, 1.0)
    # bf16 ties at the maximum share the cold mass: the draw is one of the tokens holding the maximum
    zf = rng.bf16_bits_to_f32(zc.reshape(-1)).reshape(zc.shape)
    for b in range(w.B):
        assert zf[b, cold["token"][b]] == zf[b, want["argmax"][b]]
    assert_close_log(t1["lse"], want["lse"], "lse at T=1")


def test_sample_rejects_bad_arguments():
    part = synth.zipf_partition(1000, 10, 1.1, seed=7)
    with Ctx([part]) as ctx:
        z = torch.zeros((2, 1000), dtype=torch.float32, device="cuda")
        cm = torch.ones((2, 1), dtype=torch.int32, device="cuda")
        u = torch.zeros(2, dtype=torch.float32, device="cuda")
        tok = torch.zeros(2, dtype=torch.int32, device="cuda")
        lib = cz.load_library()

        def call(inv_t=1.0, mode=cz.DENSE, uu=u, tt=tok):
            return lib.cfgzip_masked_sample(ctx.h, ctx.ids[0], None, cm.data_ptr(), 1, z.data_ptr(), cz.F32, 1000, 2, None,
                                            0, None if uu is None else uu.data_ptr(), inv_t,
                                            None if tt is None else tt.data_ptr(), None, None, None, mode, None)

        assert call() == cz.OK
        assert call(inv_t=0.0) == cz.E_ARG and call(inv_t=-1.0) == cz.E_ARG and call(inv_t=float("nan")) == cz.E_ARG
        assert call(mode=cz.SPARSE) == cz.E_ARG
        assert call(uu=None) == cz.E_ARG and call(tt=None) == cz.E_ARG
        torch.cuda.synchronize()


@pytest.mark.parametrize("config,B", [(2, 32), (3, 16), (4, 24), (5, 64)])
def test_sample_full_size_workloads(config, B):
    # full V and K of the workloads, a sample of rows, the paper's temperature 0.2
    w = synth.make_workload(config, B=B)
    cm, z, u = w.class_masks(0), w.logits(0), w.uniforms(0)
    with Ctx(w.partitions) as ctx:
        got = run_sample(ctx, w.row_part, cm, z, w.V, u, 5.0)
        near = check_sample(got, w.partitions, w.row_part, cm, z, w.V, u, 5.0, "cfg%d" % config)
    assert near <= 2


def test_sample_huge_vocabulary_many_states_per_row():
    # a long row shared by every SM: more published states than the sampling kernel keeps in registers
    V, K, B = 1000003, 500, 2
    part = synth.zipf_partition(V, K, 1.1, seed=8)
    cm = synth.class_mask_bernoulli(K, B, 0.2, rng.stream_key(81))
    z = synth.logits_normal(B, V + 5, 1.5, "f32", (82,))
    with Ctx([part]) as ctx:
        plan = cz.cfgzip_plan_query(148, 232448, V, K, B, cz.F32)
        assert plan["kind"] == 2 and plan["S"] * plan["token_warps"] + 1 > 1024  # a sampling step keeps one state per warp
        for trial in range(3):
            u = rng.uniform(rng.stream_key(83, trial), B).astype(np.float32)
            got = run_sample(ctx, None, cm, z, V, u, 3.0, stride=V + 5)
            check_sample(got, [part], None, cm, z, V, u, 3.0, "trial %d" % trial)


def test_sample_unaligned_rows_with_mixed_partitions():
    V, B, stride = 5003, 21, 5005
    parts = [synth.zipf_partition(V, K, 1.1, seed=s) for s, K in enumerate((64, 200, 31))]
    row_part = (rng.u64(rng.stream_key(91), B) % np.uint64(3)).astype(np.int32)
    cm = synth.class_mask_bernoulli(224, B, 0.3, rng.stream_key(92))
    cm[:, 0] |= 1
    z = synth.logits_normal(B, stride, 1.0, "bf16", (93,))
    u = rng.uniform(rng.stream_key(94), B).astype(np.float32)
    with Ctx(parts) as ctx:
        got = run_sample(ctx, row_part, cm, z, V, u, 5.0, stride=stride)
        check_sample(got, parts, row_part, cm, z, V, u, 5.0)
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)


@pytest.mark.parametrize("inv_t", [0.25, 1.0])
def test_sample_uniforms_at_both_ends_of_the_range_many_rows(inv_t):
    # u = 0 draws the first allowed token with weight; u just under 1 lands in the last run, where the summation
    # order of the prefix decides whether the threshold is crossed at all (if not: the last token with weight).
    # Flat distributions (high temperature) keep weight on the tail, so both cases occur across 96 rows.
    w = synth.make_workload(2, B=96)
    cm, z = w.class_masks(11), w.logits(11)
    u = np.where(np.arange(96) % 3 == 0, np.float32(0.0), np.float32(1.0) - np.float32(2.0 ** -24)).astype(np.float32)
    with Ctx(w.partitions) as ctx:
        got = run_sample(ctx, None, cm, z, w.V, u, inv_t)
        assert cz.cfgzip_poll_status(ctx.h)[1:] == (0, 0)
    check_sample(got, w.partitions, None, cm, z, w.V, u, inv_t, "1/T=%g" % inv_t)
    allowed = synth.unpack_bits(got["vocab_mask"], w.V)
    for b in range(96):
        assert allowed[b, got["token"][b]]
        if u[b] == 0.0:
            assert got["token"][b] == np.flatnonzero(allowed[b])[0]   # every allowed logit is finite: weight > 0
