"""Pins of the offline oracle (oracle/offline.py): Algorithm 1, the stack-adjacency relation of Appendix C and the
grouping of Section 3.1, against what the paper prints and against brute force on toy grammars."""
import itertools
import os

import pytest

import synth
from oracle import offline

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _grammar(name):
    names, start, prods = synth.grammars.GRAMMARS[name]()
    return names, offline.Grammar(len(names), start, prods)


def test_figure3_worked_example():
    names, g = _grammar("figure3")
    adj = offline.stack_adjacency(g)
    ix = {n: i for i, n in enumerate(names)}
    assert (ix["C"], ix["X"]) in adj            # X is popped right after C, which leaves nothing behind
    for line in open(os.path.join(ROOT, "tests", "golden", "fig3_stack_backtrack.txt")):
        if line.startswith("#") or not line.strip():
            continue
        prefix, _, s_in, s_out = line.split()
        want = (tuple(ix[ch] for ch in s_in), tuple(ix[ch] for ch in s_out.replace("-", "")))
        assert offline.displacement(g, adj, prefix.encode()) == frozenset([want]), prefix
    # without the adjacency filter the backtrack at 'x' would still find X only (one production starts with x),
    # but a token that starts inside the figure's token has its own, shorter, input stack
    assert offline.displacement(g, adj, b"bc") == frozenset([((ix["B"], ix["C"]), ())])
    assert offline.displacement(g, adj, b"zz") == frozenset()


@pytest.mark.parametrize("name", ["figure3", "arithmetic", "json_like"])
def test_adjacency_graph_search_equals_enumeration_of_parses(name):
    _, g = _grammar(name)
    by_graph = offline.stack_adjacency(g)
    by_parses = offline.stack_adjacency_by_parses(g, 9)
    assert by_parses == by_graph
    assert offline.stack_adjacency_by_parses(g, 4) <= by_graph   # short parses realise a part of it


@pytest.mark.parametrize("name", ["figure3", "arithmetic", "json_like"])
def test_algorithm1_equals_the_definition_by_brute_force(name):
    _, g = _grammar(name)
    adj = offline.stack_adjacency(g)
    chars = sorted({a for _, a, _ in g.productions})
    n_checked = n_nonempty = 0
    for n in (1, 2, 3):
        words = list(itertools.product(chars, repeat=n))
        if n == 3:
            words = words[:: max(1, len(words) // 150)]
        for w in words:
            t = bytes(w)
            got = offline.displacement(g, adj, t)
            assert got == offline.displacement_by_definition(g, adj, t), t
            n_checked += 1
            n_nonempty += bool(got)
    assert n_checked > 30 and n_nonempty > 5


def test_displacement_agrees_with_the_transition_function_from_the_start_symbol():
    # a pair ((S), beta) is in the displacement exactly when beta is reached from the stack (S) (Equation 2)
    _, g = _grammar("arithmetic")
    adj = offline.stack_adjacency(g)
    for t in (b"a", b"(a", b"a+", b"(a)", b"(a)*", b"((", b")"):
        from_start = {beta for alpha, beta in offline.displacement(g, adj, t) if alpha == (g.start,)}
        assert from_start == offline.pi(g, t, (g.start,)), t


@pytest.mark.parametrize("name", ["arithmetic", "json_like"])
def test_tokens_of_one_class_are_interchangeable(name):
    # Theorem 2 with Theorem 1: swapping a token for another of equal displacement never changes whether a
    # token sequence is a prefix of the language. Exhaustive over sequences of up to three tokens drawn from
    # the classes with several members.
    names, g = _grammar(name)
    tokens = synth.grammars.toy_vocabulary((names, g.start, g.productions), max_len=2, extra=30)
    c, r, sigs = offline.token_classes(g, tokens)
    classes = {}
    for i, k in enumerate(c):
        classes.setdefault(k, []).append(i)
    multi = [m for k, m in sorted(classes.items()) if len(m) > 1 and sigs[m[0]]]   # non-empty displacement, several members
    assert len(multi) >= 3
    pool = [m[0] for m in multi][:6] + [classes[k][0] for k in sorted(classes) if len(classes[k]) == 1][:4]
    swaps = 0
    for members in multi[:6]:
        a, others = members[0], members[1:3]
        for ctx_len in (0, 1, 2):
            for before in itertools.product(pool, repeat=ctx_len):
                for after in itertools.product(pool, repeat=min(ctx_len, 1)):
                    seq = [tokens[i] for i in before] + [tokens[a]] + [tokens[i] for i in after]
                    ok = offline.is_prefix(g, b"".join(seq))
                    for b in others:
                        seq_b = [tokens[i] for i in before] + [tokens[b]] + [tokens[i] for i in after]
                        assert offline.is_prefix(g, b"".join(seq_b)) == ok, (tokens[a], tokens[b], seq)
                        swaps += 1
    assert swaps > 500


def test_grouping_is_the_partition_by_equal_signature():
    sigs = [(1, 2), (), (1, 2), (3,), (), (1, 2, 0), (3,)]
    lens = [3, 2, 1, 5, 2, 1, 4]
    c, r = offline.group_tokens(sigs, lens)
    assert c == [0, 1, 0, 2, 1, 3, 2]            # classes in the order of their lowest token id
    assert r == [2, 1, 6, 5]                      # shortest member; the lower id among equally short ones
    for k, rep in enumerate(r):
        assert c[rep] == k
    for i, j in itertools.combinations(range(len(sigs)), 2):
        assert (c[i] == c[j]) == (sigs[i] == sigs[j])


def test_serialisation_is_injective_on_sets_of_pairs():
    a = frozenset([((1,), (2, 3)), ((1, 2), ())])
    b = frozenset([((1,), (2,)), ((3, 1, 2), ())])       # same symbols, cut differently
    assert offline.serialise(a) != offline.serialise(b)
    assert offline.serialise(a) == offline.serialise(frozenset(sorted(a, reverse=True)))
    assert offline.serialise(frozenset()) == ()


def test_toy_vocabularies_compress():
    # many tokens share a displacement (all tokens that cannot occur share the empty one): K is well below V
    for name in ("arithmetic", "json_like"):
        names, g = _grammar(name)
        tokens = synth.grammars.toy_vocabulary((names, g.start, g.productions), max_len=2, extra=30)
        c, r, _ = offline.token_classes(g, tokens)
        K = max(c) + 1
        assert 3 <= K < len(tokens) // 2 and len(r) == K
        assert all(len(tokens[r[k]]) == min(len(tokens[i]) for i in range(len(c)) if c[i] == k) for k in range(K))
