"""Thin ctypes binding of ``include/cfgzip.h``: same names, argument marshalling only.

Device buffers are passed as ``torch.Tensor`` (their ``data_ptr()`` is used), host buffers as
numpy arrays or pinned CPU tensors; raw integer addresses are accepted everywhere. Nothing is
computed here: every step of the path runs in the CUDA library. If the library cannot be
built or loaded the import of this module fails: there is no fallback.
"""
from __future__ import annotations

import ctypes
from typing import Optional, Tuple

from . import _build

F32, BF16 = 0, 1
AUTO, DENSE, SPARSE = 0, 1, 2
OK, E_ARG, E_RANGE, E_PARTITION, E_ALIGN, E_CUDA, E_NOMEM = 0, -1, -2, -3, -4, -5, -6

_vp, _i32, _i64, _int = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_int

_SIGNATURES = {
    "cfgzip_status_string": (ctypes.c_char_p, [_int]),
    "cfgzip_create": (_int, [_int, ctypes.POINTER(_vp)]),
    "cfgzip_destroy": (_int, [_vp]),
    "cfgzip_reserve_rows": (_int, [_vp, _i32]),
    "cfgzip_check_partition": (_int, [_vp, _i32, _vp, _i32]),
    "cfgzip_build_class_lists": (_int, [_vp, _i32, _i32, _vp, _vp]),
    "cfgzip_load_partition": (_int, [_vp, _vp, _i32, _vp, _i32, _vp, ctypes.POINTER(_i32)]),
    "cfgzip_free_partition": (_int, [_vp, _i32]),
    "cfgzip_expand_mask": (_int, [_vp, _i32, _vp, _vp, _i64, _vp, _i64, _i32, _int, _vp]),
    "cfgzip_mask_logits": (_int, [_vp, _vp, _int, _i64, _i32, _i32, _vp, _i64, _vp]),
    "cfgzip_masked_logsoftmax_argmax": (_int, [_vp, _i32, _vp, _vp, _i64, _vp, _int, _i64, _i32, _vp, _i64, _vp, _vp,
                                               _vp, _vp, _vp, _int, _vp]),
    "cfgzip_masked_sample": (_int, [_vp, _i32, _vp, _vp, _i64, _vp, _int, _i64, _i32, _vp, _i64, _vp, ctypes.c_float, _vp,
                                    _vp, _vp, _vp, _int, _vp]),
    "cfgzip_masked_sample_filtered": (_int, [_vp, _i32, _vp, _vp, _i64, _vp, _int, _i64, _i32, _vp, _i64, _vp, ctypes.c_float,
                                             _i32, ctypes.c_float, _vp, _vp, _vp, _vp, _int, _vp]),
    "cfgzip_multi_mask_logsoftmax_argmax": (_int, [_vp, _i32, _vp, _i64, _i32, _vp, _int, _i64, _i32, _vp, _i64, _vp, _vp, _vp,
                                                   _vp, _vp]),
    "cfgzip_plan_rows": (_int, [_vp, _i32, _vp, _i32, _vp]),
    "cfgzip_map_tokens": (_int, [_vp, _i32, _vp, _vp, _vp, _i32, _vp]),
    "cfgzip_choose_mode": (_int, [_vp, _i32, _vp, _vp, _i64, _i32, _int]),
    "cfgzip_decode_step_host": (_int, [_vp, _i32, _vp, _vp, _i64, _vp, _int, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _int,
                                       _vp]),
    "cfgzip_step_noalloc": (_int, [_vp, _i32, _vp, _i32, _vp, _i64, _vp, _int, _i64, _i32, _vp, _i64, _vp, _vp, _vp, _vp,
                                   _vp]),
    "cfgzip_rmw_floor": (_int, [_vp, _vp, _int, _i64, _i32, _i32, _vp]),
    "cfgzip_grammar_create": (_int, [_i32, _i32, _vp, _vp, _vp, _vp, _i32, ctypes.POINTER(_vp)]),
    "cfgzip_grammar_destroy": (_int, [_vp]),
    "cfgzip_grammar_adjacency": (_int, [_vp, _vp]),
    "cfgzip_displacement_signatures": (_int, [_vp, _vp, _vp, _i32, _i32, _vp, _vp, _i64]),
    "cfgzip_group_tokens": (_int, [_vp, _i32, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "cfgzip_poll_status": (_int, [_vp, _vp, ctypes.POINTER(_i32), ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
    "cfgzip_launch_count": (_int, [_vp, ctypes.POINTER(_i64)]),
    "cfgzip_set_tuning": (_int, [_vp, ctypes.c_char_p, _i32]),
    "cfgzip_plan_query": (_int, [_i32, _i32, _i32, _i32, _i32, _int, _i32, _i32, ctypes.POINTER(_i32)]),
}

EXPORTED_SYMBOLS = tuple(_SIGNATURES)

_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def load_library():
    """Build (if stale) and load ``libcfgzip.so``; raises if that is impossible."""
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


class CfgzipError(RuntimeError):
    def __init__(self, status: int, call: str):
        self.status = status
        super().__init__("%s failed: %s" % (call, cfgzip_status_string(status)))


def _check(status: int, call: str) -> None:
    if status != OK:
        raise CfgzipError(status, call)


def _ptr(x):
    """Address of a tensor / array / raw integer; None stays a null pointer."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError("cannot take the address of %r" % type(x))


def _stream(stream) -> Optional[int]:
    if stream is None:
        return None
    return stream if isinstance(stream, int) else stream.cuda_stream


def cfgzip_status_string(status: int) -> str:
    return load_library().cfgzip_status_string(status).decode()


def cfgzip_create(device: int = 0) -> int:
    """Returns the context handle (an integer address)."""
    out = _vp()
    _check(load_library().cfgzip_create(device, ctypes.byref(out)), "cfgzip_create")
    return out.value


def cfgzip_destroy(ctx: int) -> None:
    _check(load_library().cfgzip_destroy(ctx), "cfgzip_destroy")


def cfgzip_reserve_rows(ctx: int, max_rows: int) -> None:
    _check(load_library().cfgzip_reserve_rows(ctx, max_rows), "cfgzip_reserve_rows")


def cfgzip_check_partition(token_to_class, V: int, class_to_rep, K: int) -> int:
    """Returns the status code (does not raise): host-only validation."""
    return load_library().cfgzip_check_partition(_ptr(token_to_class), V, _ptr(class_to_rep), K)


def cfgzip_build_class_lists(token_to_class, V: int, K: int, off, tok) -> int:
    return load_library().cfgzip_build_class_lists(_ptr(token_to_class), V, K, _ptr(off), _ptr(tok))


def cfgzip_load_partition(ctx: int, token_to_class, V: int, class_to_rep, K: int, stream=None) -> int:
    out = _i32(-1)
    _check(load_library().cfgzip_load_partition(ctx, _ptr(token_to_class), V, _ptr(class_to_rep), K, _stream(stream),
                                                ctypes.byref(out)), "cfgzip_load_partition")
    return out.value


def cfgzip_free_partition(ctx: int, part: int) -> None:
    _check(load_library().cfgzip_free_partition(ctx, part), "cfgzip_free_partition")


def cfgzip_expand_mask(ctx: int, part0: int, row_part, class_mask, class_stride_words: int, vocab_mask,
                       vocab_stride_words: int, B: int, mode: int = AUTO, stream=None) -> None:
    _check(load_library().cfgzip_expand_mask(ctx, part0, _ptr(row_part), _ptr(class_mask), class_stride_words,
                                             _ptr(vocab_mask), vocab_stride_words, B, mode, _stream(stream)),
           "cfgzip_expand_mask")


def cfgzip_mask_logits(ctx: int, logits, dtype: int, row_stride_elems: int, B: int, V: int, vocab_mask,
                       vocab_stride_words: int, stream=None) -> None:
    _check(load_library().cfgzip_mask_logits(ctx, _ptr(logits), dtype, row_stride_elems, B, V, _ptr(vocab_mask),
                                             vocab_stride_words, _stream(stream)), "cfgzip_mask_logits")


def cfgzip_masked_logsoftmax_argmax(ctx: int, part0: int, row_part, class_mask, class_stride_words: int, logits,
                                    dtype: int, row_stride_elems: int, B: int, vocab_mask, vocab_stride_words: int,
                                    argmax, rep=None, logp_argmax=None, lse=None, logp_full=None, mode: int = AUTO,
                                    stream=None) -> None:
    _check(load_library().cfgzip_masked_logsoftmax_argmax(
        ctx, part0, _ptr(row_part), _ptr(class_mask), class_stride_words, _ptr(logits), dtype, row_stride_elems, B,
        _ptr(vocab_mask), vocab_stride_words, _ptr(argmax), _ptr(rep), _ptr(logp_argmax), _ptr(lse), _ptr(logp_full),
        mode, _stream(stream)), "cfgzip_masked_logsoftmax_argmax")


def cfgzip_masked_sample(ctx: int, part0: int, row_part, class_mask, class_stride_words: int, logits, dtype: int,
                         row_stride_elems: int, B: int, vocab_mask, vocab_stride_words: int, u, inv_temperature: float,
                         token, rep=None, logp_token=None, lse=None, mode: int = AUTO, stream=None) -> None:
    _check(load_library().cfgzip_masked_sample(
        ctx, part0, _ptr(row_part), _ptr(class_mask), class_stride_words, _ptr(logits), dtype, row_stride_elems, B,
        _ptr(vocab_mask), vocab_stride_words, _ptr(u), inv_temperature, _ptr(token), _ptr(rep), _ptr(logp_token),
        _ptr(lse), mode, _stream(stream)), "cfgzip_masked_sample")


def cfgzip_masked_sample_filtered(ctx: int, part0: int, row_part, class_mask, class_stride_words: int, logits, dtype: int,
                                  row_stride_elems: int, B: int, vocab_mask, vocab_stride_words: int, u,
                                  inv_temperature: float, top_k: int, top_p: float, token, rep=None, logp_token=None,
                                  lse=None, mode: int = AUTO, stream=None) -> None:
    _check(load_library().cfgzip_masked_sample_filtered(
        ctx, part0, _ptr(row_part), _ptr(class_mask), class_stride_words, _ptr(logits), dtype, row_stride_elems, B,
        _ptr(vocab_mask), vocab_stride_words, _ptr(u), inv_temperature, top_k, top_p, _ptr(token), _ptr(rep),
        _ptr(logp_token), _ptr(lse), mode, _stream(stream)), "cfgzip_masked_sample_filtered")


def cfgzip_multi_mask_logsoftmax_argmax(ctx: int, part0: int, class_masks, class_stride_words: int, masks_per_row: int,
                                        logits, dtype: int, row_stride_elems: int, B: int, vocab_masks,
                                        vocab_stride_words: int, argmax, rep=None, logp_argmax=None, lse=None,
                                        stream=None) -> None:
    _check(load_library().cfgzip_multi_mask_logsoftmax_argmax(
        ctx, part0, _ptr(class_masks), class_stride_words, masks_per_row, _ptr(logits), dtype, row_stride_elems, B,
        _ptr(vocab_masks), vocab_stride_words, _ptr(argmax), _ptr(rep), _ptr(logp_argmax), _ptr(lse), _stream(stream)),
        "cfgzip_multi_mask_logsoftmax_argmax")


ROWS_AS_PLANNED = 1  # pass as row_part after cfgzip_plan_rows: the kept grouping of that call is reused


def cfgzip_plan_rows(ctx: int, part0: int, row_part, B: int, stream=None) -> None:
    _check(load_library().cfgzip_plan_rows(ctx, part0, _ptr(row_part), B, _stream(stream)), "cfgzip_plan_rows")


def cfgzip_map_tokens(ctx: int, part0: int, row_part, tokens, reps, B: int, stream=None) -> None:
    _check(load_library().cfgzip_map_tokens(ctx, part0, _ptr(row_part), _ptr(tokens), _ptr(reps), B, _stream(stream)),
           "cfgzip_map_tokens")


def cfgzip_choose_mode(ctx: int, part0: int, row_part_host, class_mask_host, class_stride_words: int, B: int,
                       dtype: int) -> int:
    """DENSE or SPARSE for a batch whose class masks are in host memory (host-only, nothing is launched)."""
    mode = load_library().cfgzip_choose_mode(ctx, part0, _ptr(row_part_host), _ptr(class_mask_host), class_stride_words,
                                             B, dtype)
    if mode < 0:
        raise CfgzipError(mode, "cfgzip_choose_mode")
    return mode


def cfgzip_decode_step_host(ctx: int, part0: int, row_part_host, class_mask_host, class_stride_words: int,
                            logits_host, dtype: int, B: int, masked_logits=None, vocab_mask_host=None, argmax=None,
                            rep=None, logp_argmax=None, lse=None, mode: int = AUTO, stream=None) -> None:
    _check(load_library().cfgzip_decode_step_host(
        ctx, part0, _ptr(row_part_host), _ptr(class_mask_host), class_stride_words, _ptr(logits_host), dtype, B,
        _ptr(masked_logits), _ptr(vocab_mask_host), _ptr(argmax), _ptr(rep), _ptr(logp_argmax), _ptr(lse), mode,
        _stream(stream)), "cfgzip_decode_step_host")


def cfgzip_step_noalloc(token_to_class, V: int, class_to_rep, K: int, class_mask, class_stride_words: int, logits,
                        dtype: int, row_stride_elems: int, B: int, vocab_mask, vocab_stride_words: int, argmax,
                        rep=None, logp_argmax=None, lse=None, stream=None) -> None:
    """The fused step without a context and without any allocation (device-resident c and r, built-in scratch).

    For hosts that may not call cudaMalloc where they need the step. At most 1024 rows; runs on the
    current device; calls that could overlap on one GPU must be ordered by the caller."""
    _check(load_library().cfgzip_step_noalloc(
        _ptr(token_to_class), V, _ptr(class_to_rep), K, _ptr(class_mask), class_stride_words, _ptr(logits), dtype,
        row_stride_elems, B, _ptr(vocab_mask), vocab_stride_words, _ptr(argmax), _ptr(rep), _ptr(logp_argmax),
        _ptr(lse), _stream(stream)), "cfgzip_step_noalloc")


def cfgzip_rmw_floor(ctx: int, logits, dtype: int, row_stride_elems: int, B: int, V: int, stream=None) -> None:
    """Measurement aid: in-place sign flip of every whole 16-byte vector of the logits (one launch)."""
    _check(load_library().cfgzip_rmw_floor(ctx, _ptr(logits), dtype, row_stride_elems, B, V, _stream(stream)),
           "cfgzip_rmw_floor")


def cfgzip_grammar_create(n_nonterminals: int, start: int, prod_head, prod_terminal, prod_rhs_off, prod_rhs) -> int:
    """Grammar handle from host arrays (int32 heads, uint8 terminals, int32 offsets [n_prod + 1], int32 symbols)."""
    out = _vp()
    _check(load_library().cfgzip_grammar_create(n_nonterminals, start, _ptr(prod_head), _ptr(prod_terminal), _ptr(prod_rhs_off),
                                                _ptr(prod_rhs), len(prod_head), ctypes.byref(out)), "cfgzip_grammar_create")
    return out.value


def cfgzip_grammar_destroy(g: int) -> None:
    _check(load_library().cfgzip_grammar_destroy(g), "cfgzip_grammar_destroy")


def cfgzip_grammar_adjacency(g: int, adjacency) -> None:
    _check(load_library().cfgzip_grammar_adjacency(g, _ptr(adjacency)), "cfgzip_grammar_adjacency")


def cfgzip_displacement_signatures(g: int, token_bytes, token_off, V: int, row_words: int, signatures, signature_words=None,
                                   max_pairs: int = 1 << 20) -> int:
    """Returns the status (OK, or E_RANGE when some row did not fit); raises on argument errors."""
    rc = load_library().cfgzip_displacement_signatures(g, _ptr(token_bytes), _ptr(token_off), V, row_words, _ptr(signatures),
                                                       _ptr(signature_words), max_pairs)
    if rc not in (OK, E_RANGE):
        raise CfgzipError(rc, "cfgzip_displacement_signatures")
    return rc


def cfgzip_group_tokens(signatures, row_words: int, token_len, V: int, token_to_class, class_to_rep, n_classes, class_off=None,
                        class_tok=None, stream=None) -> None:
    _check(load_library().cfgzip_group_tokens(_ptr(signatures), row_words, _ptr(token_len), V, _ptr(token_to_class),
                                              _ptr(class_to_rep), _ptr(n_classes), _ptr(class_off), _ptr(class_tok),
                                              _stream(stream)), "cfgzip_group_tokens")


def cfgzip_poll_status(ctx: int, stream=None) -> Tuple[int, int, int]:
    """(rows with nothing allowed, token ids out of range, rows with a bad partition id) since the last poll."""
    a, b, c = _i32(0), _i32(0), _i32(0)
    _check(load_library().cfgzip_poll_status(ctx, _stream(stream), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
           "cfgzip_poll_status")
    return a.value, b.value, c.value


def cfgzip_launch_count(ctx: int) -> int:
    out = _i64(0)
    _check(load_library().cfgzip_launch_count(ctx, ctypes.byref(out)), "cfgzip_launch_count")
    return out.value


def cfgzip_set_tuning(ctx: int, name: str, value: int) -> None:
    _check(load_library().cfgzip_set_tuning(ctx, name.encode(), value), "cfgzip_set_tuning")


PLAN_FIELDS = ("kind", "groups", "S", "octets_per_block", "token_warps", "threads", "depth", "smem_bytes", "table_words",
               "stage_stride", "cm_bulk", "states_per_row", "sparse_S", "sparse_words", "state_capacity", "ctas_per_sm")


def cfgzip_plan_query(sm_count: int, smem_optin: int, V: int, K: int, B: int, dtype: int, n_partitions: int = 1,
                      aligned_class_masks: bool = True) -> dict:
    """Launch shape the library would pick for a fused dense step (host-only, no GPU)."""
    out = (_i32 * 16)()
    _check(load_library().cfgzip_plan_query(sm_count, smem_optin, V, K, B, dtype, n_partitions,
                                            1 if aligned_class_masks else 0, out), "cfgzip_plan_query")
    return dict(zip(PLAN_FIELDS, list(out)))
