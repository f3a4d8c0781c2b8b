"""cfgzip_multi_mask_logsoftmax_argmax against the CPU oracle: several class masks per logits row, the logits read
once and left unmodified. Bit-exact vocab masks, argmax and representatives; 1e-4 on the log quantities."""
import numpy as np
import pytest
import torch

import oracle
import synth
from synth import rng
from paper_2605_29986_b200 import binding as cz
from _gpu_util import Ctx, assert_close_log, dev, dtype_code, host

pytestmark = pytest.mark.gpu


def _run(ctx, cms, M, z, V, stride=None):
    B = z.shape[0]
    n = B * M
    VW = (V + 31) // 32
    stride = stride or z.shape[1]
    d_z, d_cm = dev(z), dev(cms)
    d_vm = torch.full((n, VW + 1), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    d_am = torch.full((n,), -7, dtype=torch.int32, device="cuda")
    d_rep = torch.full((n,), -7, dtype=torch.int32, device="cuda")
    d_lse = torch.full((n,), 123.0, dtype=torch.float32, device="cuda")
    d_lpa = torch.full((n,), 123.0, dtype=torch.float32, device="cuda")
    cz.cfgzip_multi_mask_logsoftmax_argmax(ctx.h, ctx.ids[0], d_cm, cms.shape[1], M, d_z, dtype_code(z), stride, B, d_vm,
                                           VW + 1, d_am, d_rep, d_lpa, d_lse, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert np.array_equal(host(d_z, z.dtype).view(np.uint8), z.view(np.uint8))      # the logits are not modified
    vm = host(d_vm, np.uint32)
    assert np.all(vm[:, VW:] == 0x5A5A5A5A)
    return dict(vocab_mask=vm[:, :VW], argmax=d_am.cpu().numpy(), rep=d_rep.cpu().numpy(), lse=d_lse.cpu().numpy(),
                logp_argmax=d_lpa.cpu().numpy())


def _compare(got, want, what):
    for key in ("vocab_mask", "argmax", "rep"):
        assert np.array_equal(got[key], want[key]), what + " " + key
    assert_close_log(got["lse"], want["lse"], what + " lse")
    assert_close_log(got["logp_argmax"], want["logp_argmax"], what + " logp_argmax")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,K,B,M", [(1, 1, 1, 1), (33, 5, 2, 3), (1000, 37, 3, 8), (4099, 130, 5, 7), (20011 + 5, 300, 9, 4),
                                     (50000, 700, 3, 32), (128256, 2048, 2, 16)])
def test_multi_mask_shapes(V, K, B, M, dtype):
    part = synth.zipf_partition(V, K, 1.1, seed=V + M)
    stride = -(-V // 8) * 8
    z = synth.logits_normal(B, stride, 2.0, dtype, (91, V, M))
    cms = synth.class_mask_bernoulli(K, B * M, 0.3, rng.stream_key(92, V, M))
    if B * M > 2:
        cms[1] = 0                                      # a (row, mask) with nothing allowed
    want = oracle.multi_mask_step(part, cms, M, np.ascontiguousarray(z[:, :V]))
    with Ctx([part]) as ctx:
        for _ in range(2):
            _compare(_run(ctx, cms, M, z, V, stride), want, "V=%d M=%d" % (V, M))
        assert cz.cfgzip_poll_status(ctx.h) == (2 * int((want["argmax"] < 0).sum()), 0, 0)


def test_multi_mask_ties_go_to_the_lowest_token_that_this_mask_allows():
    # the same spike value at three tokens of different classes: every mask must pick the lowest id IT allows
    V, K = 5000, 50
    part = synth.zipf_partition(V, K, 1.1, seed=77)
    z = synth.logits_normal(1, V, 1.0, "f32", (93,))
    spikes = [int(t) for t in (1200, 2600, 4100)]
    assert len({int(part.c[t]) for t in spikes}) == 3
    z[0, spikes] = 30.0
    bits = np.zeros((4, K), dtype=bool)
    for j, allowed in enumerate(([0, 1, 2], [1, 2], [2], [])):
        bits[j, [int(part.c[spikes[i]]) for i in allowed]] = True
        bits[j, int(part.c[0])] = True                   # and one unrelated class
    cms = synth.pack_bits(bits)
    want = oracle.multi_mask_step(part, cms, 4, z)
    with Ctx([part]) as ctx:
        got = _run(ctx, cms, 4, z, V)
    _compare(got, want, "ties")
    assert got["argmax"][:3].tolist() == spikes


def test_multi_mask_argument_errors():
    part = synth.zipf_partition(1000, 10, 1.1, seed=1)
    lib = cz.load_library()
    with Ctx([part]) as ctx:
        d_z = torch.zeros((2, 1000), dtype=torch.float32, device="cuda")
        d_cm = torch.zeros((8, 1), dtype=torch.int32, device="cuda")
        d_am = torch.zeros(8, dtype=torch.int32, device="cuda")

        def call(m=4, z=d_z, stride=1000, b=2, cms=1):
            return lib.cfgzip_multi_mask_logsoftmax_argmax(ctx.h, 0, cz._ptr(d_cm), cms, m, cz._ptr(z) if z is not None else None,
                                                           cz.F32, stride, b, None, 0, cz._ptr(d_am), None, None, None, None)

        n0 = cz.cfgzip_launch_count(ctx.h)
        assert call(m=0) == cz.E_ARG and call(z=None) == cz.E_ARG and call(stride=999) == cz.E_ARG and call(cms=0) == cz.E_ARG
        assert lib.cfgzip_multi_mask_logsoftmax_argmax(ctx.h, 0, cz._ptr(d_cm), 1, 4, cz._ptr(d_z) + 4, cz.F32, 1000, 1, None, 0,
                                                       cz._ptr(d_am), None, None, None, None) == cz.E_ALIGN
        assert call(m=20000) == cz.E_NOMEM and call(b=0) == cz.OK
        assert cz.cfgzip_launch_count(ctx.h) == n0
        assert call() == cz.OK
        torch.cuda.synchronize()
