"""cfgzip_masked_sample_filtered (top-k / top-p on the masked, tempered distribution) against the CPU oracle.

Vocab masks, masked logits and representatives are compared bit for bit. Which tokens are kept is an integer
decision: top-k is decided by order alone and must match exactly; the top-p cut is decided by sums (40-bit fixed
point on the GPU, fp64 in the oracle), so it must match wherever the oracle's target lies further than P_TOL (as a
fraction of the weight) from the cumulative weights around the cut; the few rows closer than that are only checked
for a valid draw. The drawn token must equal the oracle's unless u lies within CDF_TOL of a boundary of the CDF
over the kept tokens, where either neighbour is a valid draw. lse and logp_token: 1e-4 absolute.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from synth import rng
from paper_2605_29986_b200 import binding as cz
from _gpu_util import Ctx, assert_close_log, dev, dtype_code, host
from test_gpu_sample import check_sample

pytestmark = pytest.mark.gpu

CDF_TOL = 2e-5
P_TOL = 2e-6


def run_filtered(ctx, row_part, cm, z, V, u, inv_t, top_k, top_p, stride=None):
    B = z.shape[0]
    stride = stride or z.shape[1]
    VW = (V + 31) // 32
    d_z, d_cm, d_u = dev(z), dev(cm), dev(np.asarray(u, dtype=np.float32))
    d_rp = None if row_part is None else dev(np.asarray(row_part, dtype=np.int32))
    d_vm = torch.full((B, VW), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    d_tok = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    d_rep = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    d_lse = torch.full((B,), 123.0, dtype=torch.float32, device="cuda")
    d_lpt = torch.full((B,), 123.0, dtype=torch.float32, device="cuda")
    cz.cfgzip_masked_sample_filtered(ctx.h, ctx.ids[0], d_rp, d_cm, cm.shape[1], d_z, dtype_code(z), stride, B, d_vm, VW, d_u,
                                     inv_t, top_k, top_p, d_tok, d_rep, d_lpt, d_lse, cz.DENSE, torch.cuda.current_stream())
    torch.cuda.synchronize()
    return dict(logits=host(d_z, z.dtype), vocab_mask=host(d_vm, np.uint32), token=d_tok.cpu().numpy(),
                rep=d_rep.cpu().numpy(), lse=d_lse.cpu().numpy(), logp_token=d_lpt.cpu().numpy())


def check_filtered(got, partitions, row_part, cm, z, V, u, inv_t, top_k, top_p, what=""):
    """Returns (rows whose top-p cut is too close to call, rows drawn at a CDF boundary)."""
    zc = np.ascontiguousarray(z[:, :V]).copy()
    u64 = np.asarray(u, dtype=np.float32).astype(np.float64)
    want = oracle.sample_filtered_step(partitions, row_part, cm, zc, float(inv_t), int(top_k), float(top_p), u64, want_kept=True)
    assert np.array_equal(got["vocab_mask"], want["vocab_mask"]), what + " vocab mask"
    assert np.array_equal(got["logits"][:, :V].view(np.uint8), zc.view(np.uint8)), what + " masked logits"
    zf = rng.bf16_bits_to_f32(zc.reshape(-1)).reshape(zc.shape) if zc.dtype == np.uint16 else zc
    close_cut = near = 0
    for b in range(z.shape[0]):
        part = partitions[0 if row_part is None else int(row_part[b])]
        t, tw = int(got["token"][b]), int(want["token"][b])
        want_rep = -1 if t < 0 else int(part.r[part.c[t]])
        assert int(got["rep"][b]) == want_rep, (what, b)
        if tw < 0 or np.isneginf(want["lse"][b]):
            assert t == tw and np.isneginf(got["lse"][b]) and np.isneginf(got["logp_token"][b]), (what, b)
            continue
        allowed = (int(want["vocab_mask"][b, t // 32]) >> (t % 32)) & 1
        assert t >= 0 and allowed == 1 and np.isfinite(got["lse"][b]), (what, b, t)
        if want["p_margin"][b] <= P_TOL:
            close_cut += 1        # the cut may fall one token earlier or later: only the draw's validity is checked
            continue
        assert abs(got["lse"][b] - want["lse"][b]) <= 1e-4, (what, b, got["lse"][b], want["lse"][b])
        kept = want["kept"][b].astype(bool)
        assert kept[t], (what, b, t, "a token outside the kept set was drawn")
        lpt = float(zf[b, t]) * float(inv_t) - want["lse"][b]
        assert abs(got["logp_token"][b] - lpt) <= 1e-4, (what, b)
        if t != tw:
            w = np.where(kept, np.exp((zf[b].astype(np.float64) - zf[b][kept].max()) * inv_t), 0.0)
            cdf = np.cumsum(w) / w.sum()
            lo = cdf[t - 1] if t > 0 else 0.0
            assert cdf[t] > lo and lo - CDF_TOL <= u64[b] <= cdf[t] + CDF_TOL, (what, b, t, tw, lo, cdf[t], u64[b])
            near += 1
    return close_cut, near


FILTERS = [(1, 1.0), (3, 1.0), (50, 1.0), (0, 0.5), (0, 0.9), (0, 0.999), (40, 0.8), (100000000, 1.0), (0, 1e-6)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,K", [(1, 1), (7, 3), (33, 32), (257, 40), (1000, 37), (4099, 130)])
def test_filtered_tiny_shapes(V, K, dtype):
    part = synth.zipf_partition(V, K, 1.1, seed=V + 3)
    close = near = rows = 0
    with Ctx([part]) as ctx:
        for n, (top_k, top_p) in enumerate(FILTERS):
            B, inv_t = ((1, 1.0), (5, 5.0), (33, 0.5))[n % 3]
            cm = synth.class_mask_bernoulli(K, B, 0.5, rng.stream_key(51, V, n))
            cm[:, 0] |= 1
            z = synth.logits_normal(B, V, 2.0, dtype, (52, V, n))
            u = rng.uniform(rng.stream_key(53, V, n), B).astype(np.float32)
            got = run_filtered(ctx, None, cm, z, V, u, inv_t, top_k, top_p)
            c, m = check_filtered(got, [part], None, cm, z, V, u, inv_t, top_k, top_p, "V=%d k=%d p=%g" % (V, top_k, top_p))
            close, near, rows = close + c, near + m, rows + B
    assert close <= max(1, rows // 20) and near <= max(1, rows // 10)


def test_filtered_ties_at_the_cut_keep_the_lowest_ids():
    # bf16 logits on a coarse grid: many equal values, so both cuts fall inside groups of equal logits
    V, K, B = 6000, 60, 12
    part = synth.zipf_partition(V, K, 1.1, seed=61)
    cm = synth.class_mask_bernoulli(K, B, 0.6, rng.stream_key(62))
    zq = np.round(rng.normal_f32(rng.stream_key(63), B * V, 1.0).reshape(B, V) * 2.0) / 2.0   # steps of 0.5
    z = rng.f32_to_bf16_bits(zq.reshape(-1)).reshape(B, V)
    u = rng.uniform(rng.stream_key(64), B).astype(np.float32)
    with Ctx([part]) as ctx:
        for top_k, top_p in ((5, 1.0), (37, 1.0), (0, 0.3), (0, 0.7), (200, 0.6)):
            got = run_filtered(ctx, None, cm, z, V, u, 1.0, top_k, top_p)
            close, _ = check_filtered(got, [part], None, cm, z, V, u, 1.0, top_k, top_p, "k=%d p=%g" % (top_k, top_p))
            assert close <= 2


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_filtered_unaligned_rows_and_mixed_partitions(dtype):
    V, B, stride = 3001, 20, 3003
    parts = [synth.zipf_partition(V, K, 1.1, seed=s + 70) for s, K in enumerate((77, 64))]
    row_part = (np.arange(B) % 2).astype(np.int32)
    cm = synth.class_mask_bernoulli(77, B, 0.4, rng.stream_key(71))
    cm[:, 0] |= 1
    z = synth.logits_normal(B, stride, 1.5, dtype, (72,))
    u = rng.uniform(rng.stream_key(73), B).astype(np.float32)
    with Ctx(parts) as ctx:
        for top_k, top_p in ((10, 1.0), (0, 0.8)):
            got = run_filtered(ctx, row_part, cm, z, V, u, 2.0, top_k, top_p, stride=stride)
            check_filtered(got, parts, row_part, cm, z, V, u, 2.0, top_k, top_p)
            assert np.array_equal(got["logits"][:, V:].view(np.uint8), z[:, V:].view(np.uint8))


def test_filtered_llama_size_rows_peaked_and_flat():
    # at T = 0.2 the kept tokens are a handful (the shared-memory list serves); at T = 1 top-p needs thousands of
    # tokens, more than the list holds, and the bisection runs over the row itself
    w = synth.make_workload(2, B=32)
    cm, z, u = w.class_masks(0), w.logits(0), w.uniforms(0)
    with Ctx(w.partitions) as ctx:
        total_close = 0
        for inv_t, top_k, top_p in ((5.0, 50, 1.0), (5.0, 0, 0.9), (5.0, 40, 0.95), (1.0, 0, 0.5), (1.0, 5000, 0.9), (1.0, 3000, 1.0)):
            got = run_filtered(ctx, None, cm, z, w.V, u, inv_t, top_k, top_p)
            close, near = check_filtered(got, w.partitions, None, cm, z, w.V, u, inv_t, top_k, top_p,
                                         "1/T=%g k=%d p=%g" % (inv_t, top_k, top_p))
            total_close += close
            assert near <= 2
        assert total_close <= 3
        # twice the same call: the same bits (integer sums do not depend on the order of the addends)
        for inv_t, top_k, top_p in ((1.0, 0, 0.5), (5.0, 50, 0.9), (5.0, 2000, 1.0)):  # over the row; list, few kept; list, many kept
            a = run_filtered(ctx, None, cm, z, w.V, u, inv_t, top_k, top_p)
            b = run_filtered(ctx, None, cm, z, w.V, u, inv_t, top_k, top_p)
            for key in ("token", "lse", "logp_token"):
                assert np.array_equal(a[key].view(np.uint8), b[key].view(np.uint8)), (key, inv_t, top_k, top_p)


def test_filtered_masks_that_allow_most_of_the_vocabulary():
    # nearly every class allowed: at T = 0.2 far more tokens carry weight than the candidate list holds, so the row is
    # gone over again with a higher bar for the list and the rest is only summed; top-k / top-p that end inside the
    # list are served from it, the others (k = 5000; k beyond every token with weight and no top-p; at T = 1 a nucleus
    # of 99 %, found too large only after the search over the list) from the row
    w = synth.make_workload(2, B=8)
    cm = np.full_like(w.class_masks(0), 0xFFFFFFFF)
    cm[3, 0] &= ~np.uint32(1)
    z, u = w.logits(0), w.uniforms(0)
    with Ctx(w.partitions) as ctx:
        for inv_t, top_k, top_p in ((5.0, 50, 1.0), (5.0, 0, 0.9), (5.0, 0, 0.99), (5.0, 5000, 1.0), (5.0, 100000, 1.0),
                                    (5.0, 200, 0.5), (2.0, 20, 1.0), (1.0, 0, 0.99), (1.0, 0, 0.3)):
            got = run_filtered(ctx, None, cm, z, w.V, u, inv_t, top_k, top_p)
            close, near = check_filtered(got, w.partitions, None, cm, z, w.V, u, inv_t, top_k, top_p,
                                         "1/T=%g k=%d p=%g" % (inv_t, top_k, top_p))
            # (at T = 1 a nucleus ends among tokens of about 1e-7 of the weight each: every cut there is too close to
            # call between fixed point and fp64, and only the validity of the draw is checked)
            assert near <= 1 and (close <= 1 or inv_t < 2.0)


def test_filtered_nucleus_larger_than_the_list_found_after_the_search():
    # f32, T = 1, 18 thousand allowed tokens: the list overflows, is rebuilt with a higher bar, the search for the
    # top-p cut runs over it and finds that the list does not hold 99 % of the weight: the passes over the row take over
    V, K, B = 183926, 1426, 36
    part = synth.zipf_partition(V, K, 1.1, seed=54)
    cm = synth.class_mask_bernoulli(K, B, 0.1, rng.stream_key(91))
    cm[:, 0] |= 1
    z = synth.logits_normal(B, V + 2, 2.0, "f32", (92,))
    u = rng.uniform(rng.stream_key(93), B).astype(np.float32)
    with Ctx([part]) as ctx:
        for top_k, top_p in ((0, 0.99), (0, 0.9), (15000, 0.95)):
            got = run_filtered(ctx, None, cm, z, V, u, 1.0, top_k, top_p, stride=V + 2)
            close, near = check_filtered(got, [part], None, cm, z, V, u, 1.0, top_k, top_p, "k=%d p=%g" % (top_k, top_p))
            # (most cuts among so many light tokens are too close to call between fixed point and fp64; the rows
            # that can be called must match, and there must be some)
            assert near <= 1 and close <= B - 3, (top_k, top_p, close, near)


@pytest.mark.parametrize("B", [40, 150])
def test_filtered_one_and_two_blocks_per_row(B):
    # rows share thread-block clusters of 4 blocks up to 32 rows, of 2 up to 64, and have a block each beyond
    V, K = 9001, 200
    part = synth.zipf_partition(V, K, 1.1, seed=81)
    cm = synth.class_mask_bernoulli(K, B, 0.3, rng.stream_key(82, B))
    cm[:, 0] |= 1
    z = synth.logits_normal(B, V, 2.0, "f32", (83, B))
    u = rng.uniform(rng.stream_key(84, B), B).astype(np.float32)
    with Ctx([part]) as ctx:
        for inv_t, top_k, top_p in ((5.0, 20, 1.0), (5.0, 0, 0.9), (2.0, 300, 0.7)):
            got = run_filtered(ctx, None, cm, z, V, u, inv_t, top_k, top_p)
            close, near = check_filtered(got, [part], None, cm, z, V, u, inv_t, top_k, top_p, "B=%d k=%d p=%g" % (B, top_k, top_p))
            assert close <= 2 and near <= 2


@pytest.mark.parametrize("case", range(32))
def test_filtered_random_shapes(case):
    # shape, element type, padding, temperature, mask density, spread of the logits and both filters drawn per case
    u = rng.u64(rng.stream_key(7101, case), 12)
    V = int(u[0] % np.uint64([3000, 40000, 200000][int(u[9] % np.uint64(3))])) + 1
    K = int(u[1] % np.uint64(min(V, 5000))) + 1
    B = [1, 7, 32, 33, 64, 65, 150][int(u[2] % np.uint64(7))]
    dtype = "bf16" if u[3] & np.uint64(1) else "f32"
    pad = (-V) % 8 if (u[4] % np.uint64(4)) else 3
    inv_t = [0.5, 1.0, 5.0, 20.0][int(u[5] % np.uint64(4))]
    density = [0.01, 0.1, 0.5, 1.0][int(u[6] % np.uint64(4))]
    top_k = [0, 1, 5, 50, 300, 3000, 100000000][int(u[7] % np.uint64(7))]
    top_p = [1.0, 0.5, 0.9, 0.99, 0.1][int(u[8] % np.uint64(5))]
    if top_k == 0 and top_p == 1.0:
        top_k = 20
    sigma = [0.5, 2.0, 6.0][int(u[10] % np.uint64(3))]
    part = synth.zipf_partition(V, K, 1.1, seed=case)
    cm = synth.class_mask_bernoulli(K, B, density, rng.stream_key(7102, case))
    cm[:, 0] |= 1
    if density == 1.0:
        cm[:] = 0xFFFFFFFF
    unique = min(B, 16)
    z = np.tile(synth.logits_normal(unique, V + pad, sigma, dtype, (7103, case)), (-(-B // unique), 1))[:B]
    uu = rng.uniform(rng.stream_key(7104, case), B).astype(np.float32)
    sel = np.unique(np.linspace(0, B - 1, min(B, 12)).astype(np.int64))  # rows checked against the oracle
    what = "V=%d K=%d B=%d %s pad=%d 1/T=%g density=%g k=%d p=%g sigma=%g" % (V, K, B, dtype, pad, inv_t, density, top_k, top_p, sigma)
    with Ctx([part]) as ctx:
        got = run_filtered(ctx, None, cm, z, V, uu, inv_t, top_k, top_p, stride=V + pad)
    sub = {k: v[sel] for k, v in got.items()}
    check_filtered(sub, [part], None, cm[sel], z[sel], V, uu[sel], inv_t, top_k, top_p, what)


def test_no_filter_is_the_plain_sampling_step_and_bad_filters_are_refused():
    w = synth.make_workload(2, B=16, V=20000, K=300)
    cm, z, u = w.class_masks(1), w.logits(1), w.uniforms(1)
    lib = cz.load_library()
    with Ctx(w.partitions) as ctx:
        got = run_filtered(ctx, None, cm, z, w.V, u, 5.0, 0, 1.0)
        check_sample(got, w.partitions, None, cm, z, w.V, u, 5.0)
        d_z, d_cm, d_u = dev(z), dev(cm), dev(u)
        d_tok = torch.zeros(w.B, dtype=torch.int32, device="cuda")

        def call(k, p):
            return lib.cfgzip_masked_sample_filtered(ctx.h, 0, None, cz._ptr(d_cm), cm.shape[1], cz._ptr(d_z), cz.BF16, w.V, w.B,
                                                     None, 0, cz._ptr(d_u), 5.0, k, p, cz._ptr(d_tok), None, None, None, cz.DENSE, None)

        n0 = cz.cfgzip_launch_count(ctx.h)
        assert call(-1, 1.0) == cz.E_ARG and call(0, 0.0) == cz.E_ARG and call(0, float("nan")) == cz.E_ARG
        assert cz.cfgzip_launch_count(ctx.h) == n0
