"""Toy grammars in Greibach normal form and toy vocabularies for the offline step (inputs only).

The paper's grammars (JSON schemas, XML, C++, Bython; Section 4) and tokenizers are not available, so the
offline step is exercised on hand-written grammars of the same shape: every production is A -> a B1 .. Bn with
a one-byte terminal. A grammar is (non-terminal names, start, productions); a production is
(head index, terminal byte, tuple of non-terminal indices). Nothing here computes a displacement or a class.
"""
from __future__ import annotations

import itertools
from typing import Dict, List, Sequence, Tuple

import numpy as np

from . import rng

GrammarSpec = Tuple[List[str], int, List[Tuple[int, int, Tuple[int, ...]]]]


def _build(rules: Sequence[str], start: str) -> GrammarSpec:
    """Rules as text, "A -> a B C" (first item after the arrow is the terminal character)."""
    names: List[str] = []

    def idx(name: str) -> int:
        if name not in names:
            names.append(name)
        return names.index(name)

    idx(start)
    for rule in rules:
        idx(rule.split("->")[0].strip())
    prods = []
    for rule in rules:
        head, rhs = rule.split("->")
        items = rhs.split()
        assert len(items[0]) == 1
        prods.append((idx(head.strip()), ord(items[0]), tuple(idx(x) for x in items[1:])))
    return names, names.index(start), prods


def figure3_grammar() -> GrammarSpec:
    """The productions used in the paper's illustration of the stack backtrack (Figure 3), closed into a grammar:
    S -> s A X puts X under A, so that X is popped right after A's last symbol C."""
    return _build(["S -> s A X", "A -> a B C", "B -> b", "C -> c", "X -> x Y", "Y -> y Z J K", "Z -> z", "J -> j", "K -> k"], "S")


def arithmetic_grammar() -> GrammarSpec:
    """Sums and products of the atom 'a' with brackets."""
    return _build(["E -> a", "E -> a O E", "E -> ( E R", "E -> ( E R O E", "O -> +", "O -> *", "R -> )"], "E")


def json_like_grammar() -> GrammarSpec:
    """Nested arrays and objects over the atoms n (a number) and s (a string)."""
    return _build([
        "V -> n", "V -> s", "V -> [ A", "V -> { M",
        "A -> ]", "A -> n T", "A -> s T", "A -> [ A T", "A -> { M T",
        "T -> ]", "T -> , E",
        "E -> n T", "E -> s T", "E -> [ A T", "E -> { M T",
        "M -> }", "M -> s C",
        "C -> : W",
        "W -> n U", "W -> s U", "W -> [ A U", "W -> { M U",
        "U -> }", "U -> , P",
        "P -> s C",
    ], "V")


GRAMMARS: Dict[str, callable] = {"figure3": figure3_grammar, "arithmetic": arithmetic_grammar, "json_like": json_like_grammar}


def alphabet(spec: GrammarSpec) -> List[int]:
    return sorted({a for _, a, _ in spec[2]})


def toy_vocabulary(spec: GrammarSpec, max_len: int = 2, extra: int = 40, extra_len: int = 5, seed: int = 0) -> List[bytes]:
    """Every string of 1..max_len characters over the grammar's alphabet plus one character outside it, in a seeded
    shuffled order, followed by `extra` seeded random strings of max_len+1..extra_len characters."""
    chars = alphabet(spec) + [ord("~")]
    words = [bytes(w) for n in range(1, max_len + 1) for w in itertools.product(chars, repeat=n)]
    order = rng.permutation(rng.stream_key(rng.SEED_BASE, 77, seed), len(words))
    words = [words[i] for i in order]
    draws = rng.u64(rng.stream_key(rng.SEED_BASE, 78, seed), extra * (extra_len + 1))
    seen = set(words)
    for e in range(extra):
        n = max_len + 1 + int(draws[e * (extra_len + 1)] % np.uint64(max(1, extra_len - max_len)))
        w = bytes(chars[int(draws[e * (extra_len + 1) + 1 + j] % np.uint64(len(chars) - 1))] for j in range(n))
        if w not in seen:
            seen.add(w)
            words.append(w)
    return words
