"""GPU parity: every entry point of the C ABI against the CPU oracle, element by element.

Bit-exact for vocab masks, masked logits, argmax and representative ids; 1e-4 absolute for
the fp32-accumulated log quantities. Shapes span ragged tails (V, K not multiples of 32 or
8), several row groups and vocabulary tiles, unaligned rows, padded strides, mixed
partitions and the degenerate rows.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from synth import rng
from paper_2605_29986_b200 import binding as cz
from _gpu_util import Ctx, LOGP_TOL, compare_step, dev, dtype_code, host, oracle_step, run_fused

pytestmark = pytest.mark.gpu

TINY = [(1, 1), (31, 2), (32, 31), (33, 32), (63, 33), (64, 5), (65, 64), (1000, 37), (4099, 130)]


def _mask(K, B, p, *ids):
    return synth.class_mask_bernoulli(K, B, p, rng.stream_key(4242, *ids))


# ------------------------------------------------------------------ expand_mask

@pytest.mark.parametrize("mode", [cz.DENSE, cz.SPARSE, cz.AUTO])
@pytest.mark.parametrize("V,K", TINY)
def test_expand_tiny_shapes(V, K, mode):
    K = min(K, V)
    part = synth.zipf_partition(V, K, 1.1, seed=V)
    for B in (1, 3, 33):
        cm = _mask(K, B, 0.4, V, K, B)
        if K % 32:
            cm[:, -1] |= np.uint32((0xFFFFFFFF << (K % 32)) & 0xFFFFFFFF)  # garbage above K must be ignored
        VW = (V + 31) // 32
        with Ctx([part]) as ctx:
            d_vm = torch.full((B, VW + 2), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
            cz.cfgzip_expand_mask(ctx.h, ctx.ids[0], None, dev(cm), cm.shape[1], d_vm, VW + 2, B, mode)
            torch.cuda.synchronize()
            got = host(d_vm, np.uint32)
        assert np.array_equal(got[:, :VW], oracle.expand_mask(part.c, K, cm))
        assert np.all(got[:, VW:] == 0x5A5A5A5A)  # words past VW are never touched


@pytest.mark.parametrize("mode", [cz.DENSE, cz.SPARSE])
def test_expand_mid_size_mixed_partitions(mode):
    V, B = 20011, 70
    parts = [synth.zipf_partition(V, K, 1.1, seed=s) for s, K in enumerate((300, 257, 1024))]
    row_part = (rng.u64(rng.stream_key(1), B) % np.uint64(3)).astype(np.int32)
    KW = 32
    cm = _mask(KW * 32, B, 0.2, 7)
    want = np.stack([oracle.expand_mask(parts[row_part[b]].c, parts[row_part[b]].K, cm[b:b + 1])[0] for b in range(B)])
    with Ctx(parts) as ctx:
        d_vm = torch.zeros((B, want.shape[1]), dtype=torch.int32, device="cuda")
        cz.cfgzip_expand_mask(ctx.h, ctx.ids[0], dev(row_part), dev(cm), KW, d_vm, want.shape[1], B, mode)
        torch.cuda.synchronize()
        assert np.array_equal(host(d_vm, np.uint32), want)
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)


# ------------------------------------------------------------------ mask_logits

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,stride", [(1, 1), (7, 7), (33, 40), (1000, 1000), (1003, 1003), (4099, 4104), (20000, 20000)])
def test_mask_logits(dtype, V, stride):
    B = 5
    z = synth.logits_normal(B, stride, 1.0, dtype, (21, V))
    keep = rng.uniform(rng.stream_key(22, V), B * V).reshape(B, V) < 0.3
    keep[1] = True
    keep[2] = False
    vm = synth.pack_bits(keep)
    want = z.copy()
    oracle.mask_logits(want, V, vm)
    with Ctx([synth.identity_partition(4)]) as ctx:
        d_z = dev(z)
        cz.cfgzip_mask_logits(ctx.h, d_z, dtype_code(z), stride, B, V, dev(vm), vm.shape[1])
        cz.cfgzip_mask_logits(ctx.h, d_z, dtype_code(z), stride, B, V, dev(vm), vm.shape[1])  # idempotent
        torch.cuda.synchronize()
        assert np.array_equal(host(d_z, z.dtype).view(np.uint8), want.view(np.uint8))


def test_mask_logits_passes_non_finite_values_through():
    V = 64
    z = np.zeros((1, V), dtype=np.float32)
    z[0, 3], z[0, 4], z[0, 9] = np.inf, np.nan, -np.inf
    zb = z.view(np.uint32).copy()
    zb[0, 5] = 0x7FC12345  # NaN with a payload
    z = zb.view(np.float32)
    keep = np.ones((1, V), dtype=bool)
    keep[0, 10:20] = False
    vm = synth.pack_bits(keep)
    want = z.copy()
    oracle.mask_logits(want, V, vm)
    with Ctx([synth.identity_partition(4)]) as ctx:
        d_z = dev(z)
        cz.cfgzip_mask_logits(ctx.h, d_z, cz.F32, V, 1, V, dev(vm), vm.shape[1])
        torch.cuda.synchronize()
        assert np.array_equal(host(d_z, np.float32).view(np.uint32), want.view(np.uint32))


# ------------------------------------------------------------------ fused step

@pytest.mark.parametrize("mode", [cz.DENSE, cz.SPARSE])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,K", TINY)
def test_fused_tiny_shapes(V, K, dtype, mode):
    K = min(K, V)
    part = synth.zipf_partition(V, K, 1.1, seed=V + 1)
    for B in (1, 33):
        cm = _mask(K, B, 0.5, V, K, B, 1)
        z = synth.logits_normal(B, V, 2.0, dtype, (31, V, B))
        with Ctx([part]) as ctx:
            got = run_fused(ctx, None, cm, z, V, mode=mode, want_full=True)
        compare_step(got, oracle_step([part], None, cm, z, V, want_full=True), V, "V=%d K=%d B=%d" % (V, K, B))


@pytest.mark.parametrize("mode", [cz.DENSE, cz.SPARSE])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,stride", [(20000, 20000), (20011, 20011), (20011, 20016), (70003, 70016)])
def test_fused_several_tiles_and_ragged_tail(V, stride, dtype, mode):
    # 70 rows = two full row groups and a ragged third; V spans many 256-token tiles plus a tail;
    # stride 20011 leaves bf16/f32 rows off the 16-byte grid (scalar path), 20016 / 70016 pad them back on
    B, K = 70, 300
    part = synth.zipf_partition(V, K, 1.1, seed=5)
    cm = _mask(K, B, 0.15, V, 2)
    z = synth.logits_normal(B, stride, 2.0, dtype, (32, V))
    with Ctx([part]) as ctx:
        got = run_fused(ctx, None, cm, z, V, mode=mode, stride=stride, vm_stride=(V + 31) // 32 + 3)
    compare_step(got, oracle_step([part], None, cm, z, V), V)
    assert np.array_equal(got["logits"][:, V:].view(np.uint8), z[:, V:].view(np.uint8))  # padding untouched
    assert np.all(got["vocab_mask"][:, (V + 31) // 32:] == 0x5A5A5A5A)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("knobs", [
    dict(pipeline=0, ctas_per_sm=1), dict(pipeline=0, ctas_per_sm=4, token_warps=1, row_warps=4),
    dict(pipeline=0, ctas_per_sm=8, token_warps=2, row_warps=2), dict(pipeline=0, ctas_per_sm=2, token_warps=8, row_warps=1),
    dict(pipeline=1), dict(pipeline=1, tensor_map=0), dict(pipeline=1, pipe_warps=4, pipe_depth=2), dict(pipeline=1, pipe_warps=16, pipe_depth=3),
    dict(pipeline=1, pipe_warps=8, pipe_depth=8, ctas_per_sm=1), dict(pipeline=1, token_warps=2, row_warps=4),
    dict(pipeline=1, token_warps=1, row_warps=2, ctas_per_sm=16), dict(pipeline=1, pipe_warps=16, token_warps=16, row_warps=1),
    dict(pipeline=1, pipe_warps=4, ctas_per_sm=1, waves=2),
])
def test_fused_launch_shapes_agree(knobs, dtype):
    V, K, B = 50000, 700, 40
    part = synth.zipf_partition(V, K, 1.1, seed=6)
    cm = _mask(K, B, 0.1, 3)
    z = synth.logits_normal(B, V, 2.0, dtype, (33,))
    want = oracle_step([part], None, cm, z, V)
    with Ctx([part]) as ctx:
        for name, value in knobs.items():
            cz.cfgzip_set_tuning(ctx.h, name, value)
        for pdl in (1, 0):
            cz.cfgzip_set_tuning(ctx.h, "pdl", pdl)
            compare_step(run_fused(ctx, None, cm, z, V), want, V, "%r pdl=%d" % (knobs, pdl))
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)


def test_fused_many_chunks_per_warp():
    # enough rows and tokens that every warp of a block takes several chunks at its stride, twice in a row
    V, K, B = 200000, 900, 320
    part = synth.zipf_partition(V, K, 1.1, seed=12)
    cm = _mask(K, B, 0.1, 5)
    z = np.tile(synth.logits_normal(64, V, 2.0, "bf16", (44,)), (5, 1))
    want = oracle_step([part], None, cm, z, V)
    with Ctx([part]) as ctx:
        for _ in range(2):
            compare_step(run_fused(ctx, None, cm, z, V), want, V)
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)


@pytest.mark.parametrize("mode", [cz.DENSE, cz.SPARSE])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fused_mixed_partitions_with_different_k(dtype, mode):
    V, B = 30000, 100
    parts = [synth.zipf_partition(V, K, 1.1, seed=s) for s, K in enumerate((64, 1000, 333, 2048))]
    row_part = (rng.u64(rng.stream_key(2), B) % np.uint64(4)).astype(np.int32)
    cm = _mask(2048, B, 0.1, 9)
    z = synth.logits_normal(B, V, 1.0, dtype, (34,))
    with Ctx(parts) as ctx:
        got = run_fused(ctx, row_part, cm, z, V, mode=mode)
        assert cz.cfgzip_poll_status(ctx.h)[2] == 0
    compare_step(got, oracle_step(parts, row_part, cm, z, V), V)


@pytest.mark.parametrize("mode", [cz.DENSE, cz.SPARSE])
def test_fused_degenerate_rows_and_status(mode):
    V, K, B = 5000, 40, 6
    part = synth.zipf_partition(V, K, 1.1, seed=7)
    cm = _mask(K, B, 0.3, 11)
    cm[1] = 0                                   # nothing allowed
    cm[4] = 0
    z = synth.logits_normal(B, V, 1.0, "f32", (35,))
    only = np.zeros((1, K), dtype=bool); only[0, 5] = True
    cm[2] = synth.pack_bits(only)[0]
    z[2, part.c == 5] = -np.inf                 # allowed logits all -inf
    z[3, :] = -3.0                              # constant row: lowest allowed id
    with Ctx([part]) as ctx:
        got = run_fused(ctx, None, cm, z, V, mode=mode, want_full=True)
        assert cz.cfgzip_poll_status(ctx.h) == (2, 0, 0)
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)  # cleared by the poll
    want = oracle_step([part], None, cm, z, V, want_full=True)
    compare_step(got, want, V)
    assert got["argmax"][1] == -1 and got["rep"][1] == -1 and np.isneginf(got["lse"][1])
    assert got["argmax"][2] == np.flatnonzero(part.c == 5)[0] and np.isneginf(got["logp_argmax"][2])


@pytest.mark.parametrize("mode", [cz.DENSE, cz.SPARSE])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fused_ties_and_planted_spikes(dtype, mode):
    V, K, B = 40000, 128, 9
    part = synth.zipf_partition(V, K, 1.1, seed=8)
    bits = np.zeros((B, K), dtype=bool); bits[:, :40] = True
    cm = synth.pack_bits(bits)
    allowed = np.flatnonzero(bits[0][part.c]); masked = np.flatnonzero(~bits[0][part.c])
    zf = synth.logits_normal(B, V, 1.0, "f32", (36,))
    zf[0, allowed[100]] = 50.0
    zf[1, allowed[900]] = 50.0; zf[1, allowed[17]] = 50.0          # equal maxima -> lower id
    zf[2, masked[3]] = 99.0; zf[2, allowed[5000 % len(allowed)]] = 50.0  # spike at a masked token
    zf[3, :] = 0.0; zf[3, allowed[10]] = -0.0                        # -0.0 == +0.0
    zf[4, allowed[-1]] = 50.0                                        # last allowed token
    zf[5, allowed[0]] = 50.0
    zf[6, allowed[7]] = 50.0; zf[6, allowed[7] + 1 if allowed[7] + 1 in allowed else allowed[8]] = 50.0
    z = rng.f32_to_bf16_bits(zf.reshape(-1)).reshape(B, V) if dtype == "bf16" else zf
    with Ctx([part]) as ctx:
        got = run_fused(ctx, None, cm, z, V, mode=mode)
    want = oracle_step([part], None, cm, z, V)
    compare_step(got, want, V)
    assert got["argmax"][0] == allowed[100] and got["argmax"][1] == allowed[17] and got["argmax"][3] == allowed[0]


def test_fused_more_classes_than_the_table_path_takes():
    # K > 65535 cannot use 16-bit class ids: the generic kernel runs instead
    V, K, B = 80000, 70000, 3
    part = synth.zipf_partition(V, K, 1.1, seed=9)
    cm = _mask(K, B, 0.3, 12)
    z = synth.logits_normal(B, V, 1.0, "f32", (37,))
    with Ctx([part]) as ctx:
        got = run_fused(ctx, None, cm, z, V, want_full=True)
        d_vm = torch.zeros((B, (V + 31) // 32), dtype=torch.int32, device="cuda")
        cz.cfgzip_expand_mask(ctx.h, ctx.ids[0], None, dev(cm), cm.shape[1], d_vm, d_vm.shape[1], B, cz.DENSE)
        torch.cuda.synchronize()
    want = oracle_step([part], None, cm, z, V, want_full=True)
    compare_step(got, want, V)
    assert np.array_equal(host(d_vm, np.uint32), want["vocab_mask"])


def test_fused_without_optional_outputs_and_twice_for_determinism():
    V, K, B = 33333, 500, 37
    part = synth.zipf_partition(V, K, 1.1, seed=10)
    cm = _mask(K, B, 0.1, 13)
    z = synth.logits_normal(B, V, 2.0, "bf16", (38,))
    want = oracle_step([part], None, cm, z, V)
    with Ctx([part]) as ctx:
        d_z, d_am = dev(z), torch.empty(B, dtype=torch.int32, device="cuda")
        cz.cfgzip_masked_logsoftmax_argmax(ctx.h, ctx.ids[0], None, dev(cm), cm.shape[1], d_z, cz.BF16, V, B, None, 0,
                                           d_am)
        torch.cuda.synchronize()
        assert np.array_equal(d_am.cpu().numpy(), want["argmax"])
        assert np.array_equal(host(d_z, np.uint16), want["logits"])
        a = run_fused(ctx, None, cm, z, V)
        b = run_fused(ctx, None, cm, z, V)
    for key in ("logits", "vocab_mask", "argmax", "rep", "lse", "logp_argmax"):
        assert np.array_equal(a[key].view(np.uint8), b[key].view(np.uint8)), key


def test_fused_call_can_be_captured_in_a_cuda_graph():
    V, K, B = 128256, 2048, 32
    part = synth.zipf_partition(V, K, 1.1, seed=0, config=2)
    cm = _mask(K, B, 0.1, 14)
    z = synth.logits_normal(B, V, 2.0, "bf16", (39,))
    want = oracle_step([part], None, cm, z, V)
    with Ctx([part]) as ctx:
        d_z0, d_z, d_cm = dev(z), dev(z), dev(cm)
        d_vm = torch.zeros((B, (V + 31) // 32), dtype=torch.int32, device="cuda")
        d_am = torch.zeros(B, dtype=torch.int32, device="cuda"); d_rep = torch.zeros_like(d_am)
        d_lse = torch.zeros(B, dtype=torch.float32, device="cuda"); d_lpa = torch.zeros_like(d_lse)
        stream = torch.cuda.Stream()
        stream.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(graph, stream=stream):
                d_z.copy_(d_z0)
                cz.cfgzip_masked_logsoftmax_argmax(ctx.h, ctx.ids[0], None, d_cm, cm.shape[1], d_z, cz.BF16, V, B, d_vm,
                                                   d_vm.shape[1], d_am, d_rep, d_lpa, d_lse, None, cz.DENSE, stream)
            for _ in range(3):
                graph.replay()
        stream.synchronize()
        got = dict(logits=host(d_z, np.uint16), vocab_mask=host(d_vm, np.uint32), argmax=d_am.cpu().numpy(),
                   rep=d_rep.cpu().numpy(), lse=d_lse.cpu().numpy(), logp_argmax=d_lpa.cpu().numpy())
    compare_step(got, want, V)


# ------------------------------------------------------------------ map_tokens, host step, errors

def test_map_tokens_and_bad_ids():
    V = 9000
    parts = [synth.zipf_partition(V, 150, 1.1, seed=1), synth.zipf_partition(V, 99, 1.1, seed=2)]
    toks = np.array([0, 5, V - 1, -1, V, 77, 8999, 1234], dtype=np.int32)
    row_part = np.array([0, 1, 1, 0, 1, 0, 0, 5], dtype=np.int32)  # the last row names a partition that is not loaded
    with Ctx(parts) as ctx:
        d_out = torch.full((8,), -9, dtype=torch.int32, device="cuda")
        cz.cfgzip_map_tokens(ctx.h, ctx.ids[0], dev(row_part), dev(toks), d_out, 8)
        got = d_out.cpu().numpy()
        assert cz.cfgzip_poll_status(ctx.h) == (0, 2, 1)
        for b in range(7):
            p = parts[row_part[b]]
            assert got[b] == oracle.map_tokens(p.c, p.r, toks[b:b + 1])[0]
        assert got[7] == -9  # skipped row: untouched
        allt = np.arange(V, dtype=np.int32)
        d_all = torch.empty(V, dtype=torch.int32, device="cuda")
        cz.cfgzip_map_tokens(ctx.h, ctx.ids[1], None, dev(allt), d_all, V)
        assert np.array_equal(d_all.cpu().numpy(), oracle.map_tokens(parts[1].c, parts[1].r, allt))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_decode_step_host_buffers(dtype):
    V, K, B = 25000, 400, 20
    parts = [synth.zipf_partition(V, K, 1.1, seed=s) for s in range(2)]
    row_part = (np.arange(B) % 2).astype(np.int32)
    cm = _mask(K, B, 0.2, 15)
    z = synth.logits_normal(B, V, 1.0, dtype, (40,))
    want = oracle_step(parts, row_part, cm, z, V)
    with Ctx(parts) as ctx:
        for rp in (row_part, None):
            masked = np.empty_like(z); vm = np.empty((B, (V + 31) // 32), dtype=np.uint32)
            am = np.empty(B, dtype=np.int32); rep = np.empty(B, dtype=np.int32)
            lse = np.empty(B, dtype=np.float32); lpa = np.empty(B, dtype=np.float32)
            z_in = z.copy()
            cz.cfgzip_decode_step_host(ctx.h, ctx.ids[0], rp, cm, cm.shape[1], z_in, dtype_code(z), B, masked, vm, am,
                                       rep, lpa, lse)
            assert np.array_equal(z_in.view(np.uint8), z.view(np.uint8))  # the caller's logits are left alone
            got = dict(logits=masked, vocab_mask=vm, argmax=am, rep=rep, lse=lse, logp_argmax=lpa)
            compare_step(got, want if rp is not None else oracle_step(parts[:1], None, cm, z, V), V)


def test_argument_errors_are_reported_before_any_launch():
    V, K, B = 1000, 50, 4
    part = synth.zipf_partition(V, K, 1.1, seed=3)
    lib = cz.load_library()
    with Ctx([part]) as ctx:
        d_cm = dev(_mask(K, B, 0.5, 16)); d_z = dev(synth.logits_normal(B, V, 1.0, "f32", (41,)))
        d_vm = torch.zeros((B, 32), dtype=torch.int32, device="cuda"); d_am = torch.zeros(B, dtype=torch.int32, device="cuda")
        n0 = cz.cfgzip_launch_count(ctx.h)

        def fused(part0=0, cm=d_cm, cms=2, z=d_z, dt=cz.F32, stride=V, b=B, vm=d_vm, vms=32, am=d_am, mode=cz.DENSE,
                  full=None, lse=None):
            return lib.cfgzip_masked_logsoftmax_argmax(
                ctx.h, part0, None, cz._ptr(cm), cms, cz._ptr(z), dt, stride, b, cz._ptr(vm), vms, cz._ptr(am), None,
                None, cz._ptr(lse), cz._ptr(full), mode, None)

        assert fused(part0=3) == cz.E_RANGE and fused(part0=-1) == cz.E_RANGE
        assert fused(cm=None) == cz.E_ARG and fused(z=None) == cz.E_ARG and fused(am=None) == cz.E_ARG
        assert fused(cms=1) == cz.E_ARG and fused(stride=V - 1) == cz.E_ARG and fused(vms=31) == cz.E_ARG
        assert fused(dt=7) == cz.E_ARG and fused(mode=9) == cz.E_ARG and fused(b=-1) == cz.E_ARG
        assert fused(full=d_z) == cz.E_ARG  # logp_full needs lse
        assert fused(b=0) == cz.OK
        assert lib.cfgzip_expand_mask(ctx.h, 0, None, cz._ptr(d_cm), 2, None, 32, B, cz.DENSE, None) == cz.E_ARG
        assert lib.cfgzip_mask_logits(ctx.h, cz._ptr(d_z), cz.F32, V - 1, B, V, cz._ptr(d_vm), 32, None) == cz.E_ARG
        assert lib.cfgzip_set_tuning(ctx.h, b"nonsense", 1) == cz.E_ARG
        # the host-buffer call takes a host vector of partition ids: the "rows as planned" marker is refused, not read
        h_cm = np.zeros((B, 2), dtype=np.uint32); h_z = np.zeros((B, V), dtype=np.float32)
        assert lib.cfgzip_decode_step_host(ctx.h, 0, cz.ROWS_AS_PLANNED, h_cm.ctypes.data, 2, h_z.ctypes.data, cz.F32, B,
                                           None, None, None, None, None, None, cz.DENSE, None) == cz.E_ARG
        assert lib.cfgzip_rmw_floor(ctx.h, cz._ptr(d_z) + 4, cz.F32, V, B, V, None) == cz.E_ALIGN
        assert lib.cfgzip_rmw_floor(ctx.h, cz._ptr(d_z), cz.F32, V - 1, B, V, None) == cz.E_ARG
        assert cz.cfgzip_launch_count(ctx.h) == n0  # nothing was launched
        bad = part.c.copy(); bad[0] = K
        out = cz._i32(-1)
        import ctypes
        assert lib.cfgzip_load_partition(ctx.h, bad.ctypes.data, V, part.r.ctypes.data, K, None,
                                         ctypes.byref(out)) == cz.E_PARTITION
        cz.cfgzip_free_partition(ctx.h, ctx.ids[0])
        assert fused() == cz.E_RANGE  # freed partition
    assert lib.cfgzip_create(99, ctypes.byref(ctypes.c_void_p())) == cz.E_CUDA


def test_floor_kernel_flips_every_sign_once():
    # the measurement aid reads and rewrites every whole 16-byte vector of every row and nothing else
    V, B, stride = 1003, 5, 1008
    part = synth.zipf_partition(V, 10, 1.1, seed=5)
    with Ctx([part]) as ctx:
        for dtype, code, sign, per_vec in (("f32", cz.F32, np.uint32(0x80000000), 4), ("bf16", cz.BF16, np.uint16(0x8000), 8)):
            z = synth.logits_normal(B, stride, 1.0, dtype, (91,))
            d_z = dev(z)
            cz.cfgzip_rmw_floor(ctx.h, d_z, code, stride, B, V, torch.cuda.current_stream())
            once = host(d_z, z.dtype)
            whole = (V // per_vec) * per_vec
            bits = z.view(sign.dtype)
            assert np.array_equal(once.view(sign.dtype)[:, :whole], bits[:, :whole] ^ sign)
            assert np.array_equal(once.view(sign.dtype)[:, whole:], bits[:, whole:])   # ragged end and padding untouched
            cz.cfgzip_rmw_floor(ctx.h, d_z, code, stride, B, V, torch.cuda.current_stream())
            assert np.array_equal(host(d_z, z.dtype).view(np.uint8), z.view(np.uint8))


# ------------------------------------------------------------------ CUDA graphs

def test_steps_replayed_from_a_cuda_graph_match_the_oracle():
    # the per-step calls only enqueue work: captured once, replayed on fresh inputs, greedy and sampling
    w = synth.make_workload(2, B=40, V=20000, K=300)
    VW = (w.V + 31) // 32
    with Ctx(w.partitions) as ctx:
        d_z = torch.empty((w.B, w.V), dtype=torch.int16, device="cuda")
        d_cm = torch.empty((w.B, (w.K + 31) // 32), dtype=torch.int32, device="cuda")
        d_u = torch.empty(w.B, dtype=torch.float32, device="cuda")
        d_vm = torch.zeros((w.B, VW), dtype=torch.int32, device="cuda")
        outs = [torch.zeros(w.B, dtype=torch.int32, device="cuda") for _ in range(2)]
        outs += [torch.zeros(w.B, dtype=torch.float32, device="cuda") for _ in range(2)]
        stream = torch.cuda.Stream()
        graphs = {}
        for kind in ("greedy", "sample"):
            g = torch.cuda.CUDAGraph()
            stream.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(stream), torch.cuda.graph(g, stream=stream):
                if kind == "greedy":
                    cz.cfgzip_masked_logsoftmax_argmax(ctx.h, ctx.ids[0], None, d_cm, d_cm.shape[1], d_z, cz.BF16, w.V, w.B,
                                                       d_vm, VW, outs[0], outs[1], outs[2], outs[3], None, cz.DENSE, stream)
                else:
                    cz.cfgzip_masked_sample(ctx.h, ctx.ids[0], None, d_cm, d_cm.shape[1], d_z, cz.BF16, w.V, w.B, d_vm, VW,
                                            d_u, 5.0, outs[0], outs[1], outs[2], outs[3], cz.DENSE, stream)
            graphs[kind] = g
        for step in (0, 1, 2):
            cm, z, u = w.class_masks(step), w.logits(step), w.uniforms(step)
            for kind in ("greedy", "sample"):
                d_z.copy_(dev(z)); d_cm.copy_(dev(cm)); d_u.copy_(dev(u))
                torch.cuda.synchronize()
                graphs[kind].replay()
                torch.cuda.synchronize()
                zc = z.copy()
                if kind == "greedy":
                    want = oracle.decode_step(w.partitions, None, cm, zc)
                    assert np.array_equal(outs[0].cpu().numpy(), want["argmax"])
                    assert np.abs(outs[3].cpu().numpy() - want["lse"]).max() <= LOGP_TOL
                else:
                    want = oracle.sample_step(w.partitions, None, cm, zc, 5.0, u.astype(np.float64), want_cdf=True)
                    got = outs[0].cpu().numpy()
                    for b in np.flatnonzero(got != want["token"]):  # only within rounding of a CDF boundary
                        t = int(got[b])
                        lo = want["cdf"][b, t - 1] if t > 0 else 0.0
                        assert lo - 2e-5 <= u[b] <= want["cdf"][b, t] + 2e-5
                    assert (got != want["token"]).sum() <= 1
                assert np.array_equal(host(d_vm, np.uint32), want["vocab_mask"])
                assert np.array_equal(host(d_z, np.uint16), zc)
                part = w.partitions[0]
                tok = outs[0].cpu().numpy()
                assert np.array_equal(outs[1].cpu().numpy(), part.r[part.c[tok]])


# ------------------------------------------------------------------ kept row grouping

def test_kept_row_grouping_gives_the_same_steps_and_is_dropped_when_it_must():
    w = synth.make_workload(4, B=70, V=30000, K=700)
    VW = (w.V + 31) // 32
    lib = cz.load_library()
    with Ctx(w.partitions) as ctx:
        d_rp = dev(w.row_part)
        d_tok = torch.zeros(w.B, dtype=torch.int32, device="cuda")
        # nothing planned yet: the sentinel is an argument error
        assert lib.cfgzip_map_tokens(ctx.h, ctx.ids[0], cz.ROWS_AS_PLANNED, d_tok.data_ptr(), d_tok.data_ptr(), w.B, None) == cz.E_ARG
        cz.cfgzip_plan_rows(ctx.h, ctx.ids[0], d_rp, w.B)
        for step in range(3):
            cm, z = w.class_masks(step), w.logits(step)
            want = oracle_step(w.partitions, w.row_part, cm, z, w.V)
            d_z, d_cm = dev(z), dev(cm)
            d_vm = torch.zeros((w.B, VW), dtype=torch.int32, device="cuda")
            d_am = torch.zeros(w.B, dtype=torch.int32, device="cuda")
            d_rep = torch.zeros_like(d_am)
            d_lse = torch.zeros(w.B, dtype=torch.float32, device="cuda")
            d_lpa = torch.zeros_like(d_lse)
            before = cz.cfgzip_launch_count(ctx.h)
            cz.cfgzip_masked_logsoftmax_argmax(ctx.h, ctx.ids[0], cz.ROWS_AS_PLANNED, d_cm, cm.shape[1], d_z, cz.BF16, w.V, w.B,
                                               d_vm, VW, d_am, d_rep, d_lpa, d_lse, None, cz.DENSE)
            assert cz.cfgzip_launch_count(ctx.h) - before == 2  # streaming kernel + per-row kernel: no grouping launch
            torch.cuda.synchronize()
            got = dict(logits=host(d_z, z.dtype), vocab_mask=host(d_vm, np.uint32), argmax=d_am.cpu().numpy(),
                       rep=d_rep.cpu().numpy(), lse=d_lse.cpu().numpy(), logp_argmax=d_lpa.cpu().numpy())
            compare_step(got, want, w.V, "kept grouping, step %d" % step)
            d_map = torch.zeros_like(d_am)
            cz.cfgzip_map_tokens(ctx.h, ctx.ids[0], cz.ROWS_AS_PLANNED, d_am, d_map, w.B)
            torch.cuda.synchronize()
            assert np.array_equal(d_map.cpu().numpy(), want["rep"])
        # another batch size, or a call that regroups with an explicit vector, ends the kept grouping
        assert lib.cfgzip_map_tokens(ctx.h, ctx.ids[0], cz.ROWS_AS_PLANNED, d_tok.data_ptr(), d_tok.data_ptr(), w.B - 1, None) == cz.E_ARG
        got = run_fused(ctx, w.row_part, w.class_masks(5), w.logits(5), w.V)
        compare_step(got, oracle_step(w.partitions, w.row_part, w.class_masks(5), w.logits(5), w.V), w.V, "explicit")
        assert lib.cfgzip_map_tokens(ctx.h, ctx.ids[0], cz.ROWS_AS_PLANNED, d_tok.data_ptr(), d_tok.data_ptr(), w.B, None) == cz.E_ARG
        assert lib.cfgzip_plan_rows(ctx.h, ctx.ids[0], None, w.B, None) == cz.E_ARG
        assert cz.cfgzip_poll_status(ctx.h) == (0, 0, 0)
