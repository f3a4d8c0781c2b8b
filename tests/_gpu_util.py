"""Helpers for the GPU parity tests: device buffers via torch, calls through the C ABI binding."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import synth
from paper_2605_29986_b200 import binding as cz

LOGP_TOL = 1e-4  # absolute, on fp32-accumulated log quantities against the fp64 oracle


def dev(a: np.ndarray) -> torch.Tensor:
    """numpy -> CUDA tensor with the same bytes (uint16 / uint32 travel as int16 / int32)."""
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    elif a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t: torch.Tensor, like: np.dtype) -> np.ndarray:
    return t.cpu().numpy().view(like)


class Ctx:
    """A context with partitions loaded; destroyed on close()."""

    def __init__(self, partitions):
        self.h = cz.cfgzip_create(0)
        self.partitions = list(partitions)
        self.ids = [cz.cfgzip_load_partition(self.h, p.c, p.V, p.r, p.K) for p in self.partitions]

    def close(self):
        if self.h:
            cz.cfgzip_destroy(self.h)
            self.h = 0

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()


def dtype_code(z: np.ndarray) -> int:
    return cz.BF16 if z.dtype == np.uint16 else cz.F32


def run_fused(ctx: Ctx, row_part, cm: np.ndarray, z: np.ndarray, V: int, mode=cz.DENSE, want_vm=True, want_full=False,
              stride=None, vm_stride=None, part0=None):
    """Fused call on copies of the inputs; returns dict of numpy outputs (masked logits as the input dtype)."""
    B = z.shape[0]
    stride = stride or z.shape[1]
    VW = (V + 31) // 32
    vm_stride = vm_stride or VW
    d_z = dev(z)
    d_cm = dev(cm)
    d_rp = None if row_part is None else dev(np.asarray(row_part, dtype=np.int32))
    d_vm = torch.full((B, vm_stride), 0x5A5A5A5A, dtype=torch.int32, device="cuda") if want_vm else None
    d_am = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    d_rep = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    d_lse = torch.full((B,), 123.0, dtype=torch.float32, device="cuda")
    d_lpa = torch.full((B,), 123.0, dtype=torch.float32, device="cuda")
    d_full = torch.full((B, V), 123.0, dtype=torch.float32, device="cuda") if want_full else None
    cz.cfgzip_masked_logsoftmax_argmax(ctx.h, ctx.ids[0] if part0 is None else part0, d_rp, d_cm, cm.shape[1], d_z,
                                       dtype_code(z), stride, B, d_vm, vm_stride, d_am, d_rep, d_lpa, d_lse, d_full,
                                       mode, torch.cuda.current_stream())
    torch.cuda.synchronize()
    return dict(
        logits=host(d_z, z.dtype), vocab_mask=None if d_vm is None else host(d_vm, np.uint32),
        argmax=d_am.cpu().numpy(), rep=d_rep.cpu().numpy(), lse=d_lse.cpu().numpy(),
        logp_argmax=d_lpa.cpu().numpy(), logp_full=None if d_full is None else d_full.cpu().numpy())


def oracle_step(partitions, row_part, cm, z, V, want_full=False, threads=8):
    """Oracle on a copy; z may be wider than V (stride): only the first V columns of a row belong to it."""
    zc = np.ascontiguousarray(z[:, :V]).copy()
    out = oracle.decode_step(partitions, row_part, cm, zc, want_full=want_full, threads=threads)
    out["logits"] = zc
    return out


def assert_close_log(got: np.ndarray, want: np.ndarray, what: str):
    got = got.astype(np.float64)
    inf = np.isneginf(want)
    assert np.array_equal(np.isneginf(got), inf), what + ": -inf pattern differs"
    if (~inf).any():
        err = np.abs(got[~inf] - want[~inf]).max()
        assert err <= LOGP_TOL, "%s: max abs error %.3g > %.1g" % (what, err, LOGP_TOL)


def compare_step(got: dict, want: dict, V: int, what: str = ""):
    """Bit-exact on masks, masked logits, argmax, rep; LOGP_TOL on the log quantities."""
    if got["vocab_mask"] is not None:
        VW = (V + 31) // 32
        assert np.array_equal(got["vocab_mask"][:, :VW], want["vocab_mask"]), what + " vocab mask"
    gl = got["logits"][:, :V]
    assert np.array_equal(gl.view(np.uint8), want["logits"].view(np.uint8)), what + " masked logits"
    assert np.array_equal(got["argmax"], want["argmax"]), what + " argmax"
    assert np.array_equal(got["rep"], want["rep"]), what + " rep"
    assert_close_log(got["lse"], want["lse"], what + " lse")
    assert_close_log(got["logp_argmax"], want["logp_argmax"], what + " logp_argmax")
    if got.get("logp_full") is not None:
        assert_close_log(got["logp_full"], want["logp_full"], what + " logp_full")
