"""CPU oracle for the offline step of CFGzip: displacements of tokens under a grammar in Greibach
normal form, the stack-adjacency relation that prunes them, and the grouping of tokens with equal
displacement into classes with their representatives.

TEST INFRASTRUCTURE ONLY: plain, slow Python written from the paper (Section 2.1 for the one-state
push-down automaton of a GNF grammar, Section 3.1 "Pre-Computation" for classes, representatives and
the vectors c and r, Section 3.2 with Algorithm 1 for the displacement, Appendix B for the set it
computes, Appendix C for the stack-adjacency relation). It shares no code with the library, and the
library never imports it. Meant for toy grammars and vocabularies of a few hundred short tokens.

Conventions and readings (where the paper is silent or at odds with itself):
  - a grammar is (n_nonterminals, start, productions); a production is (head, terminal byte, rhs) with
    rhs a tuple of non-terminals; the optional production S -> epsilon plays no part in displacements
    (it consumes no character) and is not represented;
  - stacks are tuples, top first; the input queue sigma_i grows at its end;
  - Algorithm 1 tests (A_prev, A) against the adjacency relation with A_prev the symbol popped last
    (Section 3.2.2 says so, Figure 3 needs it, Appendix C computes exactly those pairs), whereas the
    set formula of Appendix B writes the test on neighbours inside the input stack; the algorithm's
    reading is taken. With A_prev = epsilon (nothing consumed yet) there is no restriction;
  - the adjacency relation is Appendix C's sub-relation: pairs (Y, Z) such that Y can be popped by a
    rule Y -> y (nothing pushed) immediately before Z is popped;
  - classes are numbered in the order of their lowest token id; the representative of a class is its
    byte-wise shortest token, the lowest id among equally short ones (the paper leaves ties open).

Parity pins (tests/test_offline_pins.py): the worked example of Figure 3, brute-force enumeration of
the definition of Appendix B on small stacks, brute-force enumeration of complete parses for the
adjacency relation, interchangeability of tokens of one class by exhaustive prefix testing
(Theorem 2 with Theorem 1), and the algebra of c and r. Nothing here is "parity unpinned".
"""
from __future__ import annotations

import itertools
from collections import deque
from typing import Dict, FrozenSet, Iterable, List, Optional, Sequence, Set, Tuple

Production = Tuple[int, int, Tuple[int, ...]]
Stack = Tuple[int, ...]
Pair = Tuple[Stack, Stack]


class Grammar:
    """A context-free grammar in Greibach normal form (Section 2.1): every production is A -> a beta."""

    def __init__(self, n_nonterminals: int, start: int, productions: Iterable[Production]):
        self.n = int(n_nonterminals)
        self.start = int(start)
        self.productions: List[Production] = [(int(h), int(a), tuple(int(x) for x in rhs)) for h, a, rhs in productions]
        for h, a, rhs in self.productions:
            assert 0 <= h < self.n and 0 <= a < 256 and all(0 <= x < self.n for x in rhs)

    def delta(self, a: int, A: int) -> List[Stack]:
        """Transition function of the one-state automaton: beta in delta(a, A) iff A -> a beta is a production."""
        return [rhs for h, t, rhs in self.productions if h == A and t == a]


# ----------------------------------------------------------------------------- Appendix C

def stack_adjacency(g: Grammar) -> Set[Tuple[int, int]]:
    """The sub-relation of Appendix C. Graph H has an edge A -> B for every production whose right-most
    non-terminal is B. For every production A -> a B_1 .. B_n Z beta (n >= 1) a breadth-first search from B_n
    finds every Y_k reachable in H (B_n included) that has a production Y_k -> y; (Y_k, Z) is adjacent."""
    edges: Dict[int, Set[int]] = {A: set() for A in range(g.n)}
    unary = set()
    for h, _, rhs in g.productions:
        if rhs:
            edges[h].add(rhs[-1])
        else:
            unary.add(h)
    rel: Set[Tuple[int, int]] = set()
    for _, _, rhs in g.productions:
        for i in range(1, len(rhs)):
            Z, start = rhs[i], rhs[i - 1]
            seen, queue = {start}, deque([start])
            while queue:
                X = queue.popleft()
                if X in unary:
                    rel.add((X, Z))
                for nxt in edges[X]:
                    if nxt not in seen:
                        seen.add(nxt)
                        queue.append(nxt)
    return rel


def stack_adjacency_by_parses(g: Grammar, max_len: int) -> Set[Tuple[int, int]]:
    """The same relation from its meaning (Section 3.2.2 with the restriction of Appendix C): run the automaton
    from the stack (S) over every string of at most max_len characters that it accepts (empty stack at the end)
    and collect (Y, Z) whenever Y is popped by a production that pushes nothing and Z is popped next."""
    rel: Set[Tuple[int, int]] = set()
    alphabet = sorted({a for _, a, _ in g.productions})

    def run(stack: Stack, steps: List[Tuple[int, bool]], left: int):
        if not stack:
            for (Y, unary), (Z, _) in zip(steps, steps[1:]):
                if unary:
                    rel.add((Y, Z))
            return
        if left == 0:
            return
        A = stack[0]
        for a in alphabet:
            for beta in g.delta(a, A):
                run(beta + stack[1:], steps + [(A, len(beta) == 0)], left - 1)

    run((g.start,), [], max_len)
    return rel


# ----------------------------------------------------------------------------- Algorithm 1

def displacement(g: Grammar, adjacency: Set[Tuple[int, int]], token: bytes) -> FrozenSet[Pair]:
    """Algorithm 1: the displacement of `token`, the set of (sigma_i, sigma_o) such that consuming the input
    stack sigma_i completely while reading the token leaves the output stack sigma_o."""

    def CD(t: bytes, s_in: Stack, s_out: Stack, a_prev: Optional[int]) -> Set[Pair]:
        Y: Set[Pair] = set()
        if len(t) == 0:
            Y.add((s_in, s_out))
        elif len(s_out) == 0:  # stack backtrack: guess the next symbol of the input stack
            for A, a, beta in g.productions:
                if a == t[0] and (a_prev is None or (a_prev, A) in adjacency):
                    Y |= CD(t[1:], s_in + (A,), beta, A)
        else:
            for beta in g.delta(t[0], s_out[0]):
                Y |= CD(t[1:], s_in, beta + s_out[1:], s_out[0])
        return Y

    return frozenset(CD(bytes(token), (), (), None))


def displacement_by_definition(g: Grammar, adjacency: Set[Tuple[int, int]], token: bytes) -> FrozenSet[Pair]:
    """The set Algorithm 1 is said to compute (Appendix B), by brute force: for EVERY input stack alpha of at most
    len(token) symbols, apply the transition function to the token as in Equation 3 (symbols of alpha carry the tag
    0, pushed symbols the tag 1), keep the results in which alpha was consumed completely (only tag 1 left), and
    drop the runs in which a symbol of alpha other than the first was popped right after a symbol it is not
    stack-adjacent to."""
    token = bytes(token)
    out: Set[Pair] = set()

    def pi_prime(t: bytes, stack: Tuple[Tuple[int, int], ...], last_popped: Optional[int]) -> List[Tuple[Tuple[int, int], ...]]:
        if len(t) == 0:
            return [stack]
        if len(stack) == 0:
            return []
        (A, tag), rest = stack[0], stack[1:]
        if tag == 0 and last_popped is not None and (last_popped, A) not in adjacency:
            return []
        res = []
        for beta in g.delta(t[0], A):
            res += pi_prime(t[1:], tuple((B, 1) for B in beta) + rest, A)
        return res

    for n in range(1, len(token) + 1):
        for alpha in itertools.product(range(g.n), repeat=n):
            for beta in pi_prime(token, tuple((A, 0) for A in alpha), None):
                if all(tag == 1 for _, tag in beta):
                    out.add((tuple(alpha), tuple(B for B, _ in beta)))
    return frozenset(out)


def pi(g: Grammar, t: bytes, alpha: Stack) -> Set[Stack]:
    """Equation 2: the stacks reached from stack alpha by reading t."""
    if len(t) == 0:
        return {alpha}
    if len(alpha) == 0:
        return set()
    res: Set[Stack] = set()
    for beta in g.delta(t[0], alpha[0]):
        res |= pi(g, t[1:], beta + alpha[1:])
    return res


def is_prefix(g: Grammar, w: bytes) -> bool:
    """w is a prefix of the language iff some stack survives reading it from (S); valid for grammars whose every
    non-terminal derives a string (each surviving stack can then be emptied)."""
    return len(pi(g, bytes(w), (g.start,))) > 0


# ----------------------------------------------------------------------------- Section 3.1, pre-computation

def serialise(disp: FrozenSet[Pair]) -> Tuple[int, ...]:
    """Canonical sequence of integers for a displacement: its pairs in sorted order, each as
    len(sigma_i), sigma_i, len(sigma_o), sigma_o; equal sets give equal sequences and vice versa."""
    flat: List[int] = []
    for s_in, s_out in sorted(disp):
        flat += [len(s_in), *s_in, len(s_out), *s_out]
    return tuple(flat)


def group_tokens(signatures: Sequence[Sequence[int]], token_lengths: Sequence[int]):
    """Section 3.1, "Pre-Computation": tokens with equal signature form a class; returns (c, r) with classes numbered
    in the order of their lowest token id and r[k] the shortest token of class k (lowest id among the shortest).
    Written as the definition: every token is compared with the classes found so far."""
    c: List[int] = []
    firsts: List[int] = []  # lowest token id of each class
    for i, sig in enumerate(signatures):
        k = -1
        for j, f in enumerate(firsts):
            if tuple(signatures[f]) == tuple(sig):
                k = j
                break
        if k < 0:
            k = len(firsts)
            firsts.append(i)
        c.append(k)
    r: List[int] = []
    for k in range(len(firsts)):
        members = [i for i in range(len(c)) if c[i] == k]
        r.append(min(members, key=lambda i: (token_lengths[i], i)))
    return c, r


def token_classes(g: Grammar, tokens: Sequence[bytes]):
    """The whole offline step for a vocabulary: adjacency, displacement of every token, grouping.
    Returns (c, r, signatures)."""
    adj = stack_adjacency(g)
    sigs = [serialise(displacement(g, adj, t)) for t in tokens]
    c, r = group_tokens(sigs, [len(t) for t in tokens])
    return c, r, sigs
