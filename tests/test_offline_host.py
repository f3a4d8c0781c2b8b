"""Host side of the offline step behind the C ABI (no GPU needed): the stack-adjacency relation and the displacement
signatures of the library against the plain Python oracle, on the toy grammars and vocabularies."""
import numpy as np
import pytest

import synth
from oracle import offline
from paper_2605_29986_b200 import binding as cz


def grammar_arrays(prods):
    head = np.array([h for h, _, _ in prods], dtype=np.int32)
    term = np.array([a for _, a, _ in prods], dtype=np.uint8)
    off = np.zeros(len(prods) + 1, dtype=np.int32)
    off[1:] = np.cumsum([len(rhs) for _, _, rhs in prods])
    rhs = np.array([x for _, _, r in prods for x in r] or [0], dtype=np.int32)
    return head, term, off, rhs


def token_arrays(tokens):
    off = np.zeros(len(tokens) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(t) for t in tokens])
    data = np.frombuffer(b"".join(tokens) or b"\0", dtype=np.uint8).copy()
    return data, off


def library_signatures(spec, tokens, row_words=64, max_pairs=1 << 20):
    names, start, prods = spec
    g = cz.cfgzip_grammar_create(len(names), start, *grammar_arrays(prods))
    try:
        adj = np.zeros((len(names), len(names)), dtype=np.uint8)
        cz.cfgzip_grammar_adjacency(g, adj)
        data, off = token_arrays(tokens)
        sig = np.full((len(tokens), row_words), -5, dtype=np.int32)
        words = np.full(len(tokens), -5, dtype=np.int32)
        rc = cz.cfgzip_displacement_signatures(g, data, off, len(tokens), row_words, sig, words, max_pairs)
    finally:
        cz.cfgzip_grammar_destroy(g)
    return adj, sig, words, rc


@pytest.mark.parametrize("name", ["figure3", "arithmetic", "json_like"])
def test_adjacency_and_signatures_match_the_oracle(name):
    spec = synth.grammars.GRAMMARS[name]()
    names, start, prods = spec
    g = offline.Grammar(len(names), start, prods)
    tokens = synth.grammars.toy_vocabulary(spec, max_len=2, extra=40) + [b""]
    adj, sig, words, rc = library_signatures(spec, tokens)
    assert rc == cz.OK
    want_adj = offline.stack_adjacency(g)
    assert {(int(y), int(z)) for y, z in zip(*np.nonzero(adj))} == want_adj
    for i, t in enumerate(tokens):
        want = offline.serialise(offline.displacement(g, want_adj, t))
        assert words[i] == len(want), t
        assert sig[i, 0] == len(want) and tuple(sig[i, 1:1 + len(want)]) == want, t
        assert not sig[i, 1 + len(want):].any()


def test_rows_that_do_not_fit_are_reported():
    spec = synth.grammars.arithmetic_grammar()
    tokens = [b"a", b"(a)", b"~"]
    _, sig, words, rc = library_signatures(spec, tokens, row_words=4)
    assert rc == cz.E_RANGE
    assert words[2] == 0 and sig[2].tolist() == [0, 0, 0, 0]      # the token that cannot occur fits: empty displacement
    assert words[0] > 3 and not sig[0].any()                      # too long for the row: zeroed, its length reported
    _, sig, words, rc = library_signatures(spec, tokens, max_pairs=1)
    assert rc == cz.E_RANGE and (words == -1).any()


def test_grammar_argument_errors():
    lib = cz.load_library()
    import ctypes
    out = ctypes.c_void_p()
    head, term, off, rhs = grammar_arrays([(0, ord("a"), (1,)), (1, ord("b"), ())])
    assert lib.cfgzip_grammar_create(2, 0, head.ctypes.data, term.ctypes.data, off.ctypes.data, rhs.ctypes.data, 2, None) == cz.E_ARG
    assert lib.cfgzip_grammar_create(0, 0, head.ctypes.data, term.ctypes.data, off.ctypes.data, rhs.ctypes.data, 2, ctypes.byref(out)) == cz.E_ARG
    assert lib.cfgzip_grammar_create(2, 2, head.ctypes.data, term.ctypes.data, off.ctypes.data, rhs.ctypes.data, 2, ctypes.byref(out)) == cz.E_ARG
    assert lib.cfgzip_grammar_create(1, 0, head.ctypes.data, term.ctypes.data, off.ctypes.data, rhs.ctypes.data, 2, ctypes.byref(out)) == cz.E_RANGE
    assert lib.cfgzip_grammar_destroy(None) == cz.E_ARG
    assert lib.cfgzip_group_tokens(None, 4, None, 3, None, None, None, None, None, None) == cz.E_ARG
    assert lib.cfgzip_group_tokens(None, 0, None, 3, None, None, None, None, None, None) == cz.E_ARG
