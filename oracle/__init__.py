"""CPU oracle for the CFGzip decode-step path: ctypes wrapper around ``cfgzip_oracle.c``.

TEST INFRASTRUCTURE ONLY. Imported by the tests, by the smoke check and by the
bench's CPU-baseline leg; the CUDA library and its Python binding never import
it, and it imports neither of them. All arithmetic is in the C file; this
module only compiles it (gcc), marshals numpy arrays and walks rows whose
partitions differ.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cfgzip_oracle.c")
_LIB = os.path.join(_HERE, "libcfgzip_oracle.so")

F32, BF16 = 0, 1
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math) next to its source; returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        for name in ("oracle_expand_mask", "oracle_build_csr", "oracle_expand_mask_csr", "oracle_mask_logits",
                     "oracle_logsoftmax_argmax", "oracle_map_tokens", "oracle_decode_step", "oracle_sample",
                     "oracle_sample_step", "oracle_multi_mask_step", "oracle_sample_filtered"):
            getattr(_lib, name).restype = None
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _u32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.uint32)


def _dtype_code(logits: np.ndarray) -> int:
    if logits.dtype == np.float32:
        return F32
    if logits.dtype == np.uint16:  # bfloat16 bit patterns
        return BF16
    raise TypeError("logits must be float32 or uint16 (bf16 bits), got %s" % logits.dtype)


def expand_mask(c, K: int, class_mask) -> np.ndarray:
    """uint32 [B, ceil(V/32)] token mask from uint32 [B, >=ceil(K/32)] class mask."""
    c = _i32(c)
    class_mask = _u32(class_mask)
    V, B = len(c), class_mask.shape[0]
    out = np.empty((B, (V + 31) // 32), dtype=np.uint32)
    _load().oracle_expand_mask(_p(c), ctypes.c_int32(V), ctypes.c_int32(K), _p(class_mask),
                               ctypes.c_int64(class_mask.shape[1]), _p(out), ctypes.c_int64(out.shape[1]),
                               ctypes.c_int32(B))
    return out


def build_csr(c, K: int):
    """(off int32 [K+1], tok int32 [V]): members of each class in ascending token id."""
    c = _i32(c)
    off = np.empty(K + 1, dtype=np.int32)
    tok = np.empty(len(c), dtype=np.int32)
    _load().oracle_build_csr(_p(c), ctypes.c_int32(len(c)), ctypes.c_int32(K), _p(off), _p(tok))
    return off, tok


def expand_mask_csr(off, tok, V: int, K: int, class_mask) -> np.ndarray:
    off, tok, class_mask = _i32(off), _i32(tok), _u32(class_mask)
    B = class_mask.shape[0]
    out = np.empty((B, (V + 31) // 32), dtype=np.uint32)
    _load().oracle_expand_mask_csr(_p(off), _p(tok), ctypes.c_int32(V), ctypes.c_int32(K), _p(class_mask),
                                   ctypes.c_int64(class_mask.shape[1]), _p(out), ctypes.c_int64(out.shape[1]),
                                   ctypes.c_int32(B))
    return out


def mask_logits(logits: np.ndarray, V: int, vocab_mask) -> None:
    """In place on a C-contiguous [B, stride] array (float32, or uint16 bf16 bits); stride >= V."""
    assert logits.flags.c_contiguous and logits.ndim == 2
    vocab_mask = _u32(vocab_mask)
    _load().oracle_mask_logits(_p(logits), ctypes.c_int(_dtype_code(logits)), ctypes.c_int64(logits.shape[1]),
                               ctypes.c_int32(logits.shape[0]), ctypes.c_int32(V), _p(vocab_mask),
                               ctypes.c_int64(vocab_mask.shape[1]))


def logsoftmax_argmax(logits: np.ndarray, V: int, vocab_mask, want_full: bool = False):
    """(argmax int32 [B], lse f64 [B], logp_argmax f64 [B], logp_full f64 [B,V] or None) from masked logits."""
    assert logits.flags.c_contiguous and logits.ndim == 2
    vocab_mask = _u32(vocab_mask)
    B = logits.shape[0]
    argmax = np.empty(B, dtype=np.int32)
    lse = np.empty(B, dtype=np.float64)
    lpa = np.empty(B, dtype=np.float64)
    full = np.empty((B, V), dtype=np.float64) if want_full else None
    _load().oracle_logsoftmax_argmax(_p(logits), ctypes.c_int(_dtype_code(logits)),
                                     ctypes.c_int64(logits.shape[1]), ctypes.c_int32(B), ctypes.c_int32(V),
                                     _p(vocab_mask), ctypes.c_int64(vocab_mask.shape[1]), _p(argmax), _p(lse),
                                     _p(lpa), _p(full))
    return argmax, lse, lpa, full


def sample(logits: np.ndarray, V: int, vocab_mask, inv_temperature: float, u, want_cdf: bool = False):
    """(token int32 [B], lse f64 [B], logp_token f64 [B], cdf f64 [B,V] or None) from masked logits and
    one uniform number per row: inverse CDF of the tempered distribution in token-id order."""
    assert logits.flags.c_contiguous and logits.ndim == 2
    vocab_mask = _u32(vocab_mask)
    B = logits.shape[0]
    u = np.ascontiguousarray(u, dtype=np.float64)
    assert u.shape == (B,)
    token = np.empty(B, dtype=np.int32)
    lse = np.empty(B, dtype=np.float64)
    lpt = np.empty(B, dtype=np.float64)
    cdf = np.empty((B, V), dtype=np.float64) if want_cdf else None
    _load().oracle_sample(_p(logits), ctypes.c_int(_dtype_code(logits)), ctypes.c_int64(logits.shape[1]),
                          ctypes.c_int32(B), ctypes.c_int32(V), _p(vocab_mask), ctypes.c_int64(vocab_mask.shape[1]),
                          ctypes.c_double(inv_temperature), _p(u), _p(token), _p(lse), _p(lpt), _p(cdf))
    return token, lse, lpt, cdf


def map_tokens(c, r, tokens) -> np.ndarray:
    c, r, tokens = _i32(c), _i32(r), _i32(tokens)
    reps = np.empty(len(tokens), dtype=np.int32)
    _load().oracle_map_tokens(_p(c), _p(r), ctypes.c_int32(len(c)), ctypes.c_int32(len(r)), _p(tokens),
                              _p(reps), ctypes.c_int32(len(tokens)))
    return reps


def _step_rows(c, r, K, class_mask, logits, V, want_full, out, rows):
    """Run oracle_decode_step on the row subset ``rows`` (all of one partition), writing into ``out``."""
    vm, am, rp, lse, lpa, full = out
    lib = _load()
    for b in rows:
        lib.oracle_decode_step(
            _p(c), _p(r), ctypes.c_int32(V), ctypes.c_int32(K), _p(class_mask[b:b + 1]),
            ctypes.c_int64(class_mask.shape[1]), _p(logits[b:b + 1]), ctypes.c_int(_dtype_code(logits)),
            ctypes.c_int64(logits.shape[1]), ctypes.c_int32(1), _p(vm[b:b + 1]), ctypes.c_int64(vm.shape[1]),
            _p(am[b:b + 1]), _p(rp[b:b + 1]), _p(lse[b:b + 1]), _p(lpa[b:b + 1]),
            _p(full[b:b + 1]) if full is not None else None)


def decode_step(partitions: Sequence, row_part, class_mask, logits: np.ndarray, want_full: bool = False,
                threads: int = 1):
    """One full step: expand, mask (in place on ``logits``), choose, normalise, map to representative.

    ``partitions`` is a sequence of objects with ``c``, ``r``, ``K``; ``row_part`` is None (all rows use
    partitions[0]) or an int array [B]. Rows are independent, so ``threads`` > 1 only splits rows over
    a thread pool for timing; the arithmetic per row is unchanged.
    Returns dict(vocab_mask, argmax, rep, lse, logp_argmax, logp_full).
    """
    assert logits.flags.c_contiguous and logits.ndim == 2
    class_mask = _u32(class_mask)
    B = logits.shape[0]
    V = len(partitions[0].c)
    cs = [_i32(p.c) for p in partitions]
    rs = [_i32(p.r) for p in partitions]
    vm = np.empty((B, (V + 31) // 32), dtype=np.uint32)
    am = np.empty(B, dtype=np.int32)
    rp = np.empty(B, dtype=np.int32)
    lse = np.empty(B, dtype=np.float64)
    lpa = np.empty(B, dtype=np.float64)
    full = np.empty((B, V), dtype=np.float64) if want_full else None
    out = (vm, am, rp, lse, lpa, full)
    part_of = np.zeros(B, dtype=np.int64) if row_part is None else np.asarray(row_part, dtype=np.int64)

    def run(rows: List[int]):
        for b in rows:
            p = int(part_of[b])
            _step_rows(cs[p], rs[p], int(partitions[p].K), class_mask, logits, V, want_full, out, [b])

    if threads <= 1 or B == 1:
        run(list(range(B)))
    else:
        chunks = [list(range(t, B, threads)) for t in range(threads)]
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(run, chunks))
    return dict(vocab_mask=vm, argmax=am, rep=rp, lse=lse, logp_argmax=lpa, logp_full=full)


def sample_step(partitions: Sequence, row_part, class_mask, logits: np.ndarray, inv_temperature: float, u,
                want_cdf: bool = False, threads: int = 1):
    """One full sampling step: expand, mask (in place on ``logits``), sample by inverse CDF at the given
    temperature with one uniform number per row, map the sampled token to its representative.
    Returns dict(vocab_mask, token, rep, lse, logp_token, cdf)."""
    assert logits.flags.c_contiguous and logits.ndim == 2
    class_mask = _u32(class_mask)
    B = logits.shape[0]
    V = len(partitions[0].c)
    cs = [_i32(p.c) for p in partitions]
    rs = [_i32(p.r) for p in partitions]
    u = np.ascontiguousarray(u, dtype=np.float64)
    vm = np.empty((B, (V + 31) // 32), dtype=np.uint32)
    tok = np.empty(B, dtype=np.int32)
    rp = np.empty(B, dtype=np.int32)
    lse = np.empty(B, dtype=np.float64)
    lpt = np.empty(B, dtype=np.float64)
    cdf = np.empty((B, V), dtype=np.float64) if want_cdf else None
    part_of = np.zeros(B, dtype=np.int64) if row_part is None else np.asarray(row_part, dtype=np.int64)
    lib = _load()

    def run(rows: List[int]):
        for b in rows:
            p = int(part_of[b])
            lib.oracle_sample_step(
                _p(cs[p]), _p(rs[p]), ctypes.c_int32(V), ctypes.c_int32(int(partitions[p].K)), _p(class_mask[b:b + 1]),
                ctypes.c_int64(class_mask.shape[1]), _p(logits[b:b + 1]), ctypes.c_int(_dtype_code(logits)),
                ctypes.c_int64(logits.shape[1]), ctypes.c_int32(1), _p(vm[b:b + 1]), ctypes.c_int64(vm.shape[1]),
                ctypes.c_double(inv_temperature), _p(u[b:b + 1]), _p(tok[b:b + 1]), _p(rp[b:b + 1]), _p(lse[b:b + 1]),
                _p(lpt[b:b + 1]), _p(cdf[b:b + 1]) if cdf is not None else None)

    if threads <= 1 or B == 1:
        run(list(range(B)))
    else:
        chunks = [list(range(t, B, threads)) for t in range(threads)]
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(run, chunks))
    return dict(vocab_mask=vm, token=tok, rep=rp, lse=lse, logp_token=lpt, cdf=cdf)


def multi_mask_step(partition, class_masks, masks_per_row: int, logits: np.ndarray):
    """Several class masks per logits row: ``class_masks`` is uint32 [B * masks_per_row, >=ceil(K/32)], entry
    (b, j) at row b * masks_per_row + j; ``logits`` [B, V] is left unchanged. Returns dict(vocab_mask, argmax, rep,
    lse, logp_argmax), every array with B * masks_per_row entries in the same order."""
    assert logits.flags.c_contiguous and logits.ndim == 2
    class_masks = _u32(class_masks)
    B, V = logits.shape[0], len(partition.c)
    n = B * masks_per_row
    assert class_masks.shape[0] == n
    c, r = _i32(partition.c), _i32(partition.r)
    vm = np.empty((n, (V + 31) // 32), dtype=np.uint32)
    am = np.empty(n, dtype=np.int32)
    rp = np.empty(n, dtype=np.int32)
    lse = np.empty(n, dtype=np.float64)
    lpa = np.empty(n, dtype=np.float64)
    _load().oracle_multi_mask_step(
        _p(c), _p(r), ctypes.c_int32(V), ctypes.c_int32(int(partition.K)), _p(class_masks),
        ctypes.c_int64(class_masks.shape[1]), ctypes.c_int32(masks_per_row), _p(logits), ctypes.c_int(_dtype_code(logits)),
        ctypes.c_int64(logits.shape[1]), ctypes.c_int32(B), _p(vm), ctypes.c_int64(vm.shape[1]), _p(am), _p(rp), _p(lse),
        _p(lpa))
    return dict(vocab_mask=vm, argmax=am, rep=rp, lse=lse, logp_argmax=lpa)


def sample_filtered(logits: np.ndarray, V: int, vocab_mask, inv_temperature: float, top_k: int, top_p: float, u,
                    want_kept: bool = False):
    """Top-k / top-p sampling from masked logits: dict(token, lse, logp_token, n_kept, p_margin, kept or None)."""
    assert logits.flags.c_contiguous and logits.ndim == 2
    vocab_mask = _u32(vocab_mask)
    B = logits.shape[0]
    u = np.ascontiguousarray(u, dtype=np.float64)
    assert u.shape == (B,)
    token = np.empty(B, dtype=np.int32)
    lse = np.empty(B, dtype=np.float64)
    lpt = np.empty(B, dtype=np.float64)
    n_kept = np.empty(B, dtype=np.int32)
    margin = np.empty(B, dtype=np.float64)
    kept = np.empty((B, V), dtype=np.uint8) if want_kept else None
    _load().oracle_sample_filtered(
        _p(logits), ctypes.c_int(_dtype_code(logits)), ctypes.c_int64(logits.shape[1]), ctypes.c_int32(B), ctypes.c_int32(V),
        _p(vocab_mask), ctypes.c_int64(vocab_mask.shape[1]), ctypes.c_double(inv_temperature), ctypes.c_int32(top_k),
        ctypes.c_double(top_p), _p(u), _p(token), _p(lse), _p(lpt), _p(n_kept), _p(margin), _p(kept))
    return dict(token=token, lse=lse, logp_token=lpt, n_kept=n_kept, p_margin=margin, kept=kept)


def sample_filtered_step(partitions: Sequence, row_part, class_mask, logits: np.ndarray, inv_temperature: float, top_k: int,
                         top_p: float, u, want_kept: bool = False):
    """One whole filtered sampling step: expand, mask (in place on ``logits``), sample among the top-k / top-p tokens,
    map the token to its representative. Returns dict(vocab_mask, token, rep, lse, logp_token, n_kept, p_margin, kept)."""
    class_mask = _u32(class_mask)
    B = logits.shape[0]
    V = len(partitions[0].c)
    part_of = np.zeros(B, dtype=np.int64) if row_part is None else np.asarray(row_part, dtype=np.int64)
    vm = np.empty((B, (V + 31) // 32), dtype=np.uint32)
    for b in range(B):
        p = partitions[int(part_of[b])]
        vm[b] = expand_mask(p.c, int(p.K), class_mask[b:b + 1])[0]
    mask_logits(logits, V, vm)
    out = sample_filtered(logits, V, vm, inv_temperature, top_k, top_p, u, want_kept)
    out["vocab_mask"] = vm
    out["rep"] = np.array([-1 if t < 0 else int(partitions[int(part_of[b])].r[partitions[int(part_of[b])].c[t]])
                           for b, t in enumerate(out["token"])], dtype=np.int32)
    return out
